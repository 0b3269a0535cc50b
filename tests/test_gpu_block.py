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


def test_block_with_the_three_separate_attention_stages():
    """The block through repq_qgemm (scores) -> repq_softmax_log2 -> repq_pv instead of the fused kernel."""
    parity.check_block("c2_deit_b", batch=3, staged_attention=True)
    parity.check_block("c4_llama7b", batch=2, D=512, H=4, MLP=1408, L=320, massive=2, staged_attention=True)
