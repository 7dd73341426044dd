"""Host logic of edgefm_prefill's contraction planner (tile shape and K split), checked without a GPU: invariants the kernels
rely on and its choices for the benchmark shapes."""
import itertools

from edgefm_synth import CONFIGS
from paper_2604_27476_b200 import edgefm_debug_prefill_plan

QKV, RESID, SWIGLU = 0, 1, 2


def shapes(cfg):
    qd = cfg.n_q_heads * cfg.head_dim
    return {"qkv": (QKV, (cfg.n_q_heads + 2 * cfg.n_kv_heads) * cfg.head_dim, cfg.hidden), "o": (RESID, cfg.hidden, qd),
            "gate_up": (SWIGLU, cfg.ffn, cfg.hidden), "down": (RESID, cfg.hidden, cfg.ffn)}


def test_planner_invariants():
    for name, T, sms in itertools.product(CONFIGS, (1, 7, 128, 129, 511, 1023, 2047), (148, 132, 16)):
        for op, (epi, N, K) in shapes(CONFIGS[name]).items():
            wide, splits = edgefm_debug_prefill_plan(epi, T, N, K, sms)
            assert wide in (0, 1) and 1 <= splits <= (8 if T <= 128 else 4)
            if epi != RESID:
                assert splits == 1, (name, op)                      # only `resid += acc` can take partial sums
            if epi == SWIGLU:
                assert wide == 1                                    # gate and up columns share one accumulator
            if splits > 1:
                kb = (K + 63) // 64
                step = 256 if wide else 128
                tiles = ((N + step - 1) // step) * ((T + 127) // 128)
                assert kb // splits >= 12                           # a unit keeps a main loop worth its fill and epilogue
                assert tiles <= sms                                 # only grids that leave SMs idle are split


def test_planner_choices_for_the_1_5b_shape():
    cfg = CONFIGS["qwen2.5-1.5b"]
    s = shapes(cfg)
    assert edgefm_debug_prefill_plan(*[s["down"][0], 2047, *s["down"][1:]], 148) == (1, 3)     # 96 wide tiles -> 288 units
    assert edgefm_debug_prefill_plan(*[s["qkv"][0], 2047, *s["qkv"][1:]], 148) == (1, 1)       # 128 wide tiles, one round
    wide, splits = edgefm_debug_prefill_plan(*[s["down"][0], 511, *s["down"][1:]], 148)
    assert splits > 1                                                                          # 48 narrow tiles alone would idle 100 SMs
    assert edgefm_debug_prefill_plan(*[s["o"][0], 511, *s["o"][1:]], 148)[1] in (1, 2)         # 24 k-blocks: at most two units
