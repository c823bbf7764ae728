"""The launch planner's choices for the benchmark shapes, checked without a GPU.

meteora_describe_plan runs host code only (with no device it plans for 148 SMs), so the decisions the measurements
rest on can be pinned here: which kernel a shape takes, how the work is split, and the special cases (two CTAs per
SM for short streams, short prefill grids, a nearly empty last wave, large ranks, shapes the tensor cores do not
take).  A change of the planner that moves one of these is then a visible change, not a silent one."""
import pytest
import torch

from paper_2405_13053_b200 import binding as mb


def plan(T, d_in, d_out, N=28, r=8, k=2, dtype=torch.bfloat16):
    return mb.meteora_describe_plan(mb.make_shape(T, d_in, d_out, N, r, k, dtype))


@pytest.fixture(autouse=True)
def no_gpu_planning_only():
    if torch.cuda.is_available():
        pytest.skip("the planner asks the device for its SM count; these pins are for the 148-SM default")


@pytest.mark.parametrize("T,per_sm", [(1, 2), (8, 2), (32, 2), (64, 2), (80, 1), (128, 1)])
def test_decode_batches_of_the_headline_shape_take_the_streamed_kernel(T, per_sm):
    p = plan(T, 4096, 4096)
    assert "path=stream_decode launches=1 main_ctas=128 row_tiles=32 ctas_per_tile=4 aux_ctas=20 aux_slices=10" in p
    assert f"ctas_per_sm={per_sm} " in p, p


def test_wide_layers_stream_with_one_cta_per_row_tile_and_one_per_sm():
    p = plan(1, 4096, 14336)
    assert "path=stream_decode" in p and "row_tiles=112 ctas_per_tile=1 " in p and "ctas_per_sm=1 " in p, p
    p = plan(64, 5120, 5120)
    assert "path=stream_decode" in p and "row_tiles=40 ctas_per_tile=3 " in p and "ctas_per_sm=1 " in p, p
    assert "ctas_per_sm=2 " in plan(32, 5120, 5120)


def test_batches_above_128_tokens_leave_the_streamed_kernel():
    # (129 - 256 tokens go to the cooperative kernel where the device confirms that its CTAs are all resident: a
    # question for the device, not answered here)
    assert "path=stream_decode" not in plan(129, 4096, 4096)
    assert "path=chain" in plan(300, 4096, 4096)


def test_prefill_on_pairs_and_the_carved_last_wave():
    p = plan(2048, 4096, 14336)                 # 448 pair tiles = 6 waves of 74 + 4
    assert "base=pairs_of_ctas pairs=444 " in p and "launches=4" in p and "tail_pairs_as_small_tiles=4" in p, p
    p = plan(2048, 4096, 4096)                  # 128 pair tiles: the second wave is three quarters full, nothing carved
    assert "base=pairs_of_ctas pairs=128 " in p and "launches=3" in p and "tail_pairs_as_small_tiles=0" in p, p


def test_short_prefill_grids_put_two_ctas_on_a_tile():
    p = plan(512, 14336, 4096)                  # long contraction axis: 256-token tiles, two CTAs each
    assert "base_ctas=128 cluster=2 tile_tokens=256 " in p, p
    p = plan(512, 4096, 1024)                   # 32 tiles of 128 tokens: two CTAs each
    assert "base_ctas=64 cluster=2 tile_tokens=128 " in p, p
    p = plan(512, 4096, 4096)                   # 128 tiles of 128 tokens fill the SMs: one CTA each
    assert "base_ctas=128 cluster=1 tile_tokens=128 " in p, p


def test_large_ranks_and_many_adapters():
    p = plan(32, 4096, 4096, r=64)              # one aux CTA per stacked tile so that the staged B rows fit
    assert "path=stream_decode" in p and "ctas_per_tile=4 aux_ctas=15 aux_slices=1 " in p, p
    p = plan(32, 4096, 4096, r=32)
    assert "path=stream_decode" in p and "ctas_per_tile=3 " in p, p
    assert "path=stream_decode" in plan(32, 4096, 4096, N=128)


def test_shapes_the_tensor_cores_do_not_take():
    assert plan(32, 4096, 4096, dtype=torch.float32) == "path=simt" or "path=simt" in plan(32, 4096, 4096, dtype=torch.float32)
    assert "path=simt" in plan(33, 60, 50, N=6, r=4)            # d_in no multiple of 8
    assert "path=stream_decode" in plan(30, 512, 384, r=4)      # rank 4 on the tensor cores, padded to 8
