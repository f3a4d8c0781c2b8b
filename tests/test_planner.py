"""Launch planner of the fused dense step, checked on the host over many shapes (no GPU).

Whatever the shape, the plan must stay inside the device's limits (shared memory per block, threads per
block, state scratch) and cover the whole vocabulary: a plan that does not would fault or skip tokens on
the GPU, so it is caught here first.
"""
import itertools

import pytest

from paper_2605_29986_b200 import binding as cz

SMS, SMEM = 148, 232448  # B200: SMs, opt-in shared memory per block


def _check(V, K, B, dtype, parts):
    p = cz.cfgzip_plan_query(SMS, SMEM, V, K, B, dtype, parts, True)
    n_oct = 4 * ((V + 31) // 32)
    groups_min = (B + 31) // 32
    assert p["groups"] >= groups_min
    if p["kind"] == 0:
        return p
    assert 32 <= p["threads"] <= (512 if p["kind"] == 2 else 256) and p["threads"] % 32 == 0
    assert p["threads"] % (32 * p["token_warps"]) == 0
    assert p["smem_bytes"] <= SMEM - 1024
    assert p["table_words"] >= 32 * ((K + 31) // 32 + 1)
    assert p["states_per_row"] in (p["S"], p["S"] * p["token_warps"] + 1)  # one per block (merged in the block) or per warp
    assert p["groups"] * 32 * p["states_per_row"] <= p["state_capacity"]
    assert p["S"] >= 1
    if p["kind"] == 1:
        assert p["S"] * p["octets_per_block"] >= n_oct  # contiguous ranges cover the row
    if p["kind"] == 2:
        assert p["depth"] >= 2
        if p["cm_bulk"]:
            assert p["stage_stride"] % 4 == 0 and (p["stage_stride"] // 4) % 2 == 1 and p["stage_stride"] >= (K + 31) // 32
    if p["sparse_S"]:
        assert p["sparse_S"] * p["sparse_words"] >= (V + 31) // 32 and 4 * p["sparse_words"] <= SMEM - 4096
    return p


@pytest.mark.parametrize("dtype", [cz.F32, cz.BF16])
def test_plans_stay_inside_the_device_limits(dtype):
    Vs = [1, 7, 8, 33, 255, 256, 257, 1000, 4099, 32000, 128256, 151936, 256000, 1000003]
    Ks = [1, 2, 31, 32, 33, 256, 2048, 4096, 16384, 40000, 65535, 65536, 70000]
    Bs = [1, 2, 7, 8, 9, 31, 32, 33, 100, 128, 1024, 4095, 16384]
    n = 0
    for V, K, B in itertools.product(Vs, Ks, Bs):
        if K > V:
            continue
        for parts in (1, 8):
            _check(V, K, B, dtype, parts)
            n += 1
    assert n > 1000


def test_plans_of_the_five_workloads():
    p = _check(128256, 2048, 32, cz.BF16, 1)
    assert p["kind"] == 2 and p["groups"] == 1 and p["S"] == SMS and p["cm_bulk"] == 1  # one block per SM
    p = _check(256000, 16384, 256, cz.BF16, 8)
    assert p["kind"] == 2 and p["groups"] == 16 and p["cm_bulk"] == 1
    p = _check(128256, 512, 1024, cz.F32, 1)
    assert p["kind"] == 2 and p["groups"] == 32 and p["sparse_S"] == 1
    assert _check(80000, 70000, 3, cz.F32, 1)["kind"] == 0  # 16-bit class ids impossible: per-row kernel


def test_plan_query_rejects_nonsense():
    out = (cz._i32 * 16)()
    lib = cz.load_library()
    assert lib.cfgzip_plan_query(148, 232448, 100, 200, 1, cz.F32, 1, 1, out) == cz.E_ARG
    assert lib.cfgzip_plan_query(148, 232448, 100, 10, 0, cz.F32, 1, 1, out) == cz.E_ARG
    assert lib.cfgzip_plan_query(148, 232448, 100, 10, 1, 7, 1, 1, out) == cz.E_ARG
    assert lib.cfgzip_plan_query(148, 232448, 100, 10, 1, cz.F32, 1, 1, None) == cz.E_ARG
