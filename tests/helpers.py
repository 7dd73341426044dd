"""Shared helpers of the GPU parity tests: build both sides from the same seeded host buffers."""
from __future__ import annotations

import numpy as np

from edgefm_synth import CONFIGS, GLOBAL_SEED, first_token, make_kv, make_weights

LOGIT_MAX_ABS = 3e-2      # tolerances of the benchmark spec
LOGIT_REL_L2 = 1e-2
TOKEN_MARGIN = 0.1


def top2_margin(logits: np.ndarray) -> float:
    part = np.partition(logits, -2)[-2:]
    return float(part[1] - part[0])


def compare_logits(gpu: np.ndarray, ref: np.ndarray):
    g = gpu.astype(np.float64)
    r = ref.astype(np.float64)
    max_abs = float(np.abs(g - r).max())
    rel_l2 = float(np.linalg.norm(g - r) / max(np.linalg.norm(r), 1e-30))
    return max_abs, rel_l2


def assert_logits_close(gpu, ref, what=""):
    assert np.isfinite(gpu).all(), f"{what}: non-finite logits"
    max_abs, rel_l2 = compare_logits(gpu, ref)
    assert max_abs <= LOGIT_MAX_ABS, f"{what}: max-abs {max_abs}"
    assert rel_l2 <= LOGIT_REL_L2, f"{what}: rel-L2 {rel_l2}"
    return max_abs, rel_l2


def bf16_ulp_distance(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    """Distance in bf16 steps between two arrays of bf16 bit patterns (sign-magnitude -> ordered ints)."""
    def key(x):
        x = x.astype(np.int32)
        return np.where(x & 0x8000, -(x & 0x7FFF), x & 0x7FFF)
    return np.abs(key(a_bits) - key(b_bits))


def assert_appended_rows_close(gpu_bits: np.ndarray, ref_bits: np.ndarray):
    """Appended K/V rows: the CUDA path sums in fp32, the oracle in fp64, so a value may land on the
    neighbouring bf16 code.  Allowed: one bf16 step of the value's magnitude, or 1e-3 of the tensor's
    RMS for values near zero (where a bf16 step is far below the fp32 summation error that the residual
    stream has accumulated over the layers), and almost all codes equal."""
    g = (gpu_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    r = (ref_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    assert np.isfinite(g).all()
    step = np.maximum(np.abs(r) * 2.0 ** -7, 1e-3 * float(np.sqrt(np.mean(r * r))))
    assert np.all(np.abs(g - r) <= step), float(np.max(np.abs(g - r) / step))
    assert np.mean(gpu_bits == ref_bits) > 0.97


class Pair:
    """The oracle model and the CUDA context fed from the same host weights and KV prefix."""

    def __init__(self, cfg, seed=GLOBAL_SEED, cache_len=None, max_context=None, weights=None, kv_format=None, block_tokens=0):
        import torch
        from oracle import OracleModel
        from paper_2604_27476_b200 import DecodeContext, upload_weights

        self.cfg = cfg
        self.T0 = cfg.cache_len if cache_len is None else cache_len
        self.max_context = max_context or (self.T0 + cfg.steps)
        self.weights = weights if weights is not None else make_weights(cfg, seed)
        self.k, self.v = make_kv(cfg, seed, self.T0)
        self.oracle = OracleModel(cfg, self.weights, self.max_context, kv_format=kv_format or "bf16")
        if self.T0:
            self.oracle.load_kv(self.k, self.v)
        self.ptrs, self.keep = upload_weights(self.weights)
        self.ctx = DecodeContext(cfg, self.ptrs, self.max_context, kv_format=kv_format, block_tokens=block_tokens)
        self.kd = torch.from_numpy(self.k.view(np.int16)).cuda()
        self.vd = torch.from_numpy(self.v.view(np.int16)).cuda()
        if self.T0:
            self.ctx.prefill_kv(self.kd, self.vd)
        torch.cuda.synchronize()

    def close(self):
        self.ctx.close()
        self.oracle.close()
