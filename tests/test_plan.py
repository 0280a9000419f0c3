"""Host-side planning of the statistics kernels (no GPU): for every batch size the chosen tile
shape must respect the rules the kernels and the TMA unit rely on -- 16-byte box rows, 128-byte
aligned shared-memory destinations, at most 256 rows per box, the ring inside the shared-memory
limit, enough row slots per thread, and exact row counts where a kernel variant assumes them."""
import pytest

import paper_2406_13936_b200 as pkg

SMEM = 232448          # opt-in shared memory per CTA on sm_100


def check_plan(dtype, b, p):
    lpr = p["lanes_per_row"]
    row_bytes = 16 * lpr
    assert p["smem_bytes"] <= SMEM and p["stages"] >= 2
    assert lpr in (1, 2, 4, 8, 16, 32)
    assert 1 <= p["box_rows"] <= 256
    assert p["box_rows"] * p["row_boxes"] >= p["rows_per_cta"]
    assert p["stage_bytes"] % 128 == 0                       # every ring buffer starts 128-byte aligned
    if p["row_boxes"] > 1:
        assert (p["box_rows"] * row_bytes) % 128 == 0        # so does every stacked box
    if p["boxes_per_stage"] > 1:
        assert (p["stage_bytes"] // p["boxes_per_stage"]) % 128 == 0
    if p["route"] == 0:
        assert dtype == "bf16" and 7 <= b <= 32 and p["box_rows"] == b
        return
    if p["route"] == 4:
        # tcgen05 Gram kernel: k-blocks of 128-byte rows, each k-block on a 1024-byte boundary.
        # b <= 128: 1..3 column segments of ceil8(b) rows stacked, at most 128 operand rows, 4 k-blocks
        # per stage; b > 128: two row blocks of 128, 2 k-blocks per stage.
        assert dtype == "bf16" and 32 < b <= 256
        rows_blk = (b + 7) // 8 * 8
        mblocks = 1 if b <= 128 else 2
        if mblocks == 1:
            assert p["box_rows"] == (128 // rows_blk) * rows_blk and p["boxes_per_stage"] == 4
        else:
            assert p["box_rows"] == rows_blk and p["boxes_per_stage"] == 2
        assert lpr == 8 and p["rows_per_cta"] == b
        assert p["stage_bytes"] == p["boxes_per_stage"] * p["box_rows"] * 128
        assert (p["stage_bytes"] // p["boxes_per_stage"]) % 1024 == 0
        # the operand descriptors (128 rows per row block) of the last k-block stay inside the allocation
        assert p["stages"] * p["stage_bytes"] + (128 * mblocks - p["box_rows"]) * 128 + 1024 <= p["smem_bytes"]
        return
    groups = p["warps_per_box"] * 32 // lpr                  # row groups that share a box
    R = p["rows_per_thread"]
    assert R * groups >= p["rows_per_cta"]
    if p["keep_in_registers"]:
        assert R <= 16
        if p["route"] == 2:
            # the single-CTA kernel predicates only a thread's last row: all others must exist
            assert (R - 1) * groups < b
    else:
        assert R <= 32
    if p["full"]:
        assert R * groups == p["rows_per_cta"]
    assert p["warps_per_box"] * p["boxes_per_stage"] == 8
    if p["route"] == 1:
        C = p["cluster_size"]
        assert 2 <= C <= 8 and p["rows_per_cta"] * C >= b and p["rows_per_cta"] <= 512
        assert (C - 1) * p["rows_per_cta"] < b               # no CTA of the cluster is left without rows
        assert row_bytes >= 128
        if p["full"]:
            assert b % C == 0
    else:
        assert p["cluster_size"] == 1 and p["rows_per_cta"] == b


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_every_batch_size_gets_a_valid_plan(dtype):
    for b in range(2, 4097):
        p = pkg.plan_stats(dtype, b)
        if dtype == "bf16" and 7 <= b <= 32:
            assert p["route"] == 0
        elif dtype == "bf16" and 32 < b <= 256:
            assert p["route"] == 4
        elif b > 256:
            assert p["route"] == 1
        else:
            assert p["route"] == 2
        check_plan(dtype, b, p)


def test_routes_outside_the_fast_path():
    assert pkg.plan_stats("f32", 64, aligned=False)["route"] == 3
    assert pkg.plan_stats("f32", 5000)["route"] == 3
    assert pkg.plan_stats("bf16", 100000)["route"] == 3


def test_documented_shapes():
    p = pkg.plan_stats("f32", 256)
    assert (p["lanes_per_row"], p["rows_per_thread"], p["full"], p["stage_bytes"]) == (16, 16, 1, 65536)
    p = pkg.plan_stats("f32", 64)
    assert (p["lanes_per_row"], p["boxes_per_stage"], p["rows_per_thread"]) == (32, 2, 16)
    p = pkg.plan_stats("f32", 1024)
    assert (p["cluster_size"], p["rows_per_cta"], p["lanes_per_row"], p["full"]) == (4, 256, 16, 1)
    p = pkg.plan_stats("f32", 4096)
    assert (p["cluster_size"], p["rows_per_cta"], p["lanes_per_row"]) == (8, 512, 8)
    p = pkg.plan_stats("bf16", 16)
    assert (p["route"], p["boxes_per_stage"], p["lanes_per_row"]) == (0, 8, 32)
    p = pkg.plan_stats("bf16", 128)
    assert (p["route"], p["stages"], p["stage_bytes"]) == (4, 3, 65536)
    p = pkg.plan_stats("bf16", 33)
    assert (p["route"], p["stages"], p["box_rows"]) == (4, 3, 120)
    p = pkg.plan_stats("bf16", 256)
    assert (p["route"], p["stages"], p["stage_bytes"], p["boxes_per_stage"]) == (4, 3, 65536, 2)
