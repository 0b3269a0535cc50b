"""Free-running parity of repq_block_forward against the oracle's block on the seeded workloads."""
import pytest

from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2402_05628_b200.build import build_library
    build_library()


def test_block_c1_vit_s_fp32():
    rel, mx = parity.check_block("c1_vit_s", batch=1)
    print("c1 rel_l2 %.3e max_abs %.3e" % (rel, mx))


def test_block_c2_deit_b_small_batch():
    parity.check_block("c2_deit_b", batch=3)


def test_block_c2_w6a6_small_batch():
    parity.check_block("c2_deit_b_w6a6", batch=2)


def test_block_c2_bf16_output():
    parity.check_block("c2_deit_b", batch=2, out_dtype="bf16")


def test_block_c2_full_batch_sampled_items():
    parity.check_block("c2_deit_b", batch=64, sample_items=(0, 31, 63))


def test_block_c3_vit_l_sampled():
    parity.check_block("c3_vit_l", batch=4, sample_items=(0, 3))


def test_block_causal_8bit_log_codes_small():
    # LLaMA-shaped semantics (causal Softmax, 8-bit log codes, head dim 128) at a CPU-sized width
    parity.check_block("c4_llama7b", batch=2, D=512, H=4, MLP=1408, L=320, massive=2)


def test_block_c3_full_batch_sampled_items():
    parity.check_block("c3_vit_l", batch=32, sample_items=(0, 31))


def test_block_c4_llama_shaped_full_size_sampled_item():
    # full LLaMA-7B-shaped layer (batch 4 x 2048 tokens, dim 4096, MLP 11008, causal, 8-bit log codes);
    # the oracle recomputes one batch item
    parity.check_block("c4_llama7b", batch=4, sample_items=(3,))


def test_block_llama_form_small():
    # RMS normalisation, rotary embedding on Q / K, gated SiLU MLP, causal Softmax with 8-bit log codes
    parity.check_block("c4_llama7b_arch", batch=2, D=512, H=4, MLP=1408, L=320, massive=2)
    parity.check_block("c4_llama7b_arch", batch=2, D=512, H=8, MLP=1408, L=200, massive=2, out_dtype="bf16")


def test_block_c4_llama_form_full_size_sampled_item():
    parity.check_block("c4_llama7b_arch", batch=4, sample_items=(1,))


@pytest.mark.parametrize("name,overrides", [
    ("c2_deit_b", {}), ("c2_deit_b_w6a6", {}), ("c3_vit_l", {}),
    ("c4_llama7b", dict(D=1024, H=8, MLP=2816, L=640, massive=4)),
    ("c4_llama7b_arch", dict(D=1024, H=8, MLP=2816, L=640, massive=4)),
])
def test_block_stages_teacher_forced_on_workload_tensors(name, overrides):
    """Each stage of the block on the workload's own distributions, fed the oracle's output of the stage before:
    every in-block code tensor against the oracle's."""
    rep = parity.check_block_teacher_forced(name, **overrides)
    print(name, rep)


def test_block_stages_teacher_forced_c4_full_size():
    parity.check_block_teacher_forced("c4_llama7b")


def test_block_stages_teacher_forced_c4_llama_form_full_size():
    parity.check_block_teacher_forced("c4_llama7b_arch")


@pytest.mark.parametrize("name,batch,overrides", [
    ("c1_vit_s", 4, {}), ("c4_llama7b_arch", 2, dict(D=512, H=4, MLP=1408, L=320, massive=2)),
])
def test_calibration_pipeline_matches_oracle(name, batch, overrides):
    """Algorithm 1 for one block (dual clipping for the LayerNorm activations, percentile calibration elsewhere,
    round-to-nearest weights) through the library against the oracle's pipeline."""
    parity.check_calibration(name, batch, **overrides)


def test_block_with_byte_wide_weight_storage():
    """Weights kept one code per byte in device memory or packed (4-bit: two per byte, 6-bit: four to three bytes):
    the same block output, bit for bit."""
    import numpy as np
    import torch
    from paper_2402_05628_b200.engine import QuantBlock
    from workloads import make_block_inputs
    for name, ratio in (("c2_deit_b", 2.0), ("c2_deit_b_w6a6", 4.0 / 3.0)):
        w = make_block_inputs(name, batch=3)
        a, b = QuantBlock(w, weight_storage="packed"), QuantBlock(w, weight_storage="bytes")
        assert a.qkv.codes.shape[1] * ratio == b.qkv.codes.shape[1]
        x = torch.from_numpy(np.ascontiguousarray(w.x)).to(a.device).to(a.act_dtype)
        ya, yb = a.forward(x), b.forward(x)
        torch.cuda.synchronize()
        assert torch.equal(ya, yb)


def test_block_with_the_three_separate_attention_stages():
    """The block through repq_qgemm (scores) -> repq_softmax_log2 -> repq_pv instead of the fused kernel."""
    parity.check_block("c2_deit_b", batch=3, staged_attention=True)
    parity.check_block("c4_llama7b", batch=2, D=512, H=4, MLP=1408, L=320, massive=2, staged_attention=True)


def test_block_forward_host_matches_the_device_path():
    """Host-buffer entry point: five batches (two of them from the same host buffer) pipelined through two
    staging buffers give, batch by batch, the bits that repq_block_forward gives on device buffers; the device
    path itself is checked against the oracle above."""
    import numpy as np
    import torch
    from paper_2402_05628_b200.engine import QuantBlock
    from paper_2402_05628_b200 import binding as B
    from workloads import make_block_inputs

    w = make_block_inputs("c2_deit_b", batch=2)
    blk = QuantBlock(w)
    rng = np.random.default_rng(5)
    xs = [torch.from_numpy(np.ascontiguousarray(w.x * s)).to(blk.act_dtype).pin_memory()
          for s in (1.0, 0.5, 1.5, float(rng.uniform(0.7, 1.3)))]
    x_host = [xs[0], xs[1], xs[2], xs[1], xs[3]]
    y_host = [torch.zeros(xs[0].shape, dtype=blk.out_dtype).pin_memory() for _ in x_host]
    blk.forward_host(x_host, y_host)
    torch.cuda.synchronize()
    assert B.repq_device_status() == 0
    for xh, yh in zip(x_host, y_host):
        y_dev = blk.forward(xh.to(blk.device))
        torch.cuda.synchronize()
        assert torch.equal(y_dev.cpu(), yh)
    assert not torch.equal(y_host[0], y_host[1])
    # pageable host memory: the copies no longer overlap, the results are the same
    xp = [xs[2].clone(), xs[0].clone(), xs[3].clone()]
    yp = [torch.zeros(xs[0].shape, dtype=blk.out_dtype) for _ in xp]
    blk.forward_host(xp, yp)
    torch.cuda.synchronize()
    assert torch.equal(yp[0], y_host[2]) and torch.equal(yp[1], y_host[0]) and torch.equal(yp[2], y_host[4])
    # nothing to do, and arguments that cannot work
    d, p = blk.desc(2), blk.params()
    ws = blk.workspace(2)
    B.repq_block_forward_host(d, p, [], [], blk._staging[0], blk._staging[1], ws)
    same = blk._staging[0][0]
    with pytest.raises(B.RepqError):
        B.repq_block_forward_host(d, p, x_host[:1], y_host[:1], [same, same], blk._staging[1], ws)
    torch.cuda.synchronize()


def test_block_back_to_back_passes_are_identical():
    """Twenty passes queued without a synchronisation in between (each kernel's prologue overlaps the tail of the
    kernel before) write the same bits as a pass that runs alone."""
    import numpy as np
    import torch
    from paper_2402_05628_b200.engine import QuantBlock
    from paper_2402_05628_b200 import binding as B
    from workloads import make_block_inputs

    for name, batch in (("c2_deit_b", 8), ("c1_vit_s", 1)):
        w = make_block_inputs(name, batch=batch)
        blk = QuantBlock(w)
        x = torch.from_numpy(np.ascontiguousarray(w.x)).to(blk.device).to(blk.act_dtype)
        alone = blk.forward(x).clone()
        torch.cuda.synchronize()
        outs = [torch.empty_like(alone) for _ in range(20)]
        for y in outs:
            blk.forward(x, y)
        torch.cuda.synchronize()
        assert B.repq_device_status() == 0
        for y in outs:
            assert torch.equal(y, alone)
