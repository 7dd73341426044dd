"""The host-side tile schedule of the weight stream (no GPU needed): for every operator shape of the five configurations,
every ring-slot size the launch plan can choose and both warp counts of the kernel builds, the tiles must cover every
(unit, 256-column piece) exactly once, stay inside a head for the QKV operator, fit the slot, use at most four box heights,
and the partial-sum slots of a unit block must be consecutive and complete."""
import numpy as np
import pytest

from edgefm_synth import CONFIGS

PH_QKV, PH_RESID, PH_SWIGLU, PH_LMHEAD = 0, 1, 2, 3


def operator_shapes(cfg):
    H, F, d = cfg.hidden, cfg.ffn, cfg.head_dim
    return [(PH_QKV, cfg.qkv_rows // 2, H, d // 2, 0), (PH_RESID, H, cfg.n_q_heads * d, 0, 1), (PH_SWIGLU, F, H, 0, 2),
            (PH_RESID, H, F, 0, 3), (PH_LMHEAD, cfg.vocab, H, 0, 4)]


def check_operator(kind, units, K, head_half, op_index, n_ctas, n_warps, slot_rows):
    from paper_2604_27476_b200 import edgefm_debug_plan_operator
    plan = edgefm_debug_plan_operator(kind, units, K, head_half, op_index, n_ctas, n_warps, slot_rows)
    paired = kind in (PH_QKV, PH_SWIGLU)
    nkb = (K + 255) // 256
    assert 1 <= len(plan["variant_rows"]) <= 4
    covered = np.zeros((units, nkb), np.int32)
    for c in range(n_ctas):
        slots_seen = {}
        for w in range(n_warps):
            run_open = False
            for t in plan["tiles"][c][w]:
                m, v0, u0 = t["m"], t["v0"], t["unit_base"]
                assert t["op"] == op_index and 1 <= m <= (8 if paired else 16) and m * (2 if paired else 1) <= slot_rows
                assert plan["variant_rows"][t["variant"]] == m
                assert 0 <= v0 < m and u0 + m <= units and t["kcol"] < nkb
                if kind == PH_QKV:
                    assert u0 // head_half == (u0 + m - 1) // head_half          # a block never crosses a head
                assert t["first"] == (not run_open)                                # accumulators restart exactly at run starts
                run_open = not t["flush"]
                covered[u0 + v0:u0 + m, t["kcol"]] += 1
                if t["flush"] and not t["direct"]:
                    slots_seen.setdefault((u0, m, v0), []).append(t["slot"])
            assert not run_open                                                     # every run ends with a flush
        # partial slots of a block: consecutive, and exactly what its combine entry says
        comb = {(e["unit_base"], e["m"], e["v0"]): e for e in plan["combines"][c]}
        assert set(comb) == set(slots_seen)
        for key, e in comb.items():
            assert sorted(slots_seen[key]) == list(range(e["first_slot"], e["first_slot"] + e["n_slots"]))
            assert e["first_slot"] + e["n_slots"] <= 48
    assert (covered == 1).all(), (np.argwhere(covered != 1)[:5], covered.min(), covered.max())
    counts = [sum(len(l) for l in plan["tiles"][c]) for c in range(n_ctas)]
    return max(counts)


@pytest.mark.parametrize("name", sorted(CONFIGS))
def test_schedule_covers_every_weight_exactly_once(name):
    cfg = CONFIGS[name]
    for n_warps in (11, 7):
        for slot_rows in (4, 6, 10, 12, 14, 16):
            for shape in operator_shapes(cfg):
                check_operator(*shape, 148, n_warps, slot_rows)


def test_schedule_odd_shapes_and_small_grids():
    # rows not divisible by anything convenient, K with a ragged last piece, fewer units than CTAs
    for kind, units, K, hh, op in [(PH_RESID, 7, 40, 0, 1), (PH_LMHEAD, 1, 264, 0, 4), (PH_SWIGLU, 43, 520, 0, 2), (PH_QKV, 96, 72, 32, 0),
                                   (PH_RESID, 3001, 1000, 0, 3), (PH_LMHEAD, 152064, 3584, 0, 4)]:
        for n_ctas in (1, 5, 148):
            check_operator(kind, units, K, hh, op, n_ctas, 11, 16)
