"""Second, structurally different definition of the decoder: numpy fp64, no KV cache.

TEST INFRASTRUCTURE ONLY.  `full_forward` recomputes causal attention over the whole token prefix
from scratch (O(T^2)), which is the plain definition that KV-cached decoding only accelerates
(Eq. 1-4 of the paper: y_t depends on all previous tokens; the cache is an implementation detail).
It is used to pin the C++ oracle's cache indexing, position handling and GQA mapping on small
models.  It keeps the same rounding points as the oracle where they are observable: k (after RoPE)
and v are rounded to bf16 before being attended, and inter-operator vectors are rounded to fp32.
"""
from __future__ import annotations

import numpy as np


def _bf16_bits_to_f64(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _round_bf16(x64: np.ndarray) -> np.ndarray:
    """fp64 -> fp32 -> bf16 (RNE) -> fp64, via integer arithmetic on the fp32 bit pattern."""
    u = x64.astype(np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16 << 16
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def _f32(x64: np.ndarray) -> np.ndarray:
    return x64.astype(np.float32).astype(np.float64)


def _rms(x, w, eps):
    return _f32(x * (1.0 / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)) * w)


def _rope_all(u, positions, theta):
    """u [T][heads][d] -> rotated; pairs (i, i+d/2)."""
    d = u.shape[-1]
    inv = theta ** (-2.0 * np.arange(d // 2) / d)
    phi = np.asarray(positions, np.float64)[:, None] * inv[None, :]            # [T][d/2]
    c, s = np.cos(phi)[:, None, :], np.sin(phi)[:, None, :]
    a, b = u[..., : d // 2], u[..., d // 2:]
    return _f32(np.concatenate([a * c - b * s, b * c + a * s], axis=-1))


def _int8_rows(x64: np.ndarray) -> np.ndarray:
    """Compression of Sec. 3.9 as the oracle reads it, written with numpy fp32 array operations: per row (last axis)
    scale = amax / 127, code = clip(rint(x * (127 / amax))), value seen by attention = code * scale."""
    x = x64.astype(np.float32)
    amax = np.abs(x).max(axis=-1, keepdims=True)
    safe = np.where(amax > 0, amax, np.float32(1))
    codes = np.clip(np.rint(x * (np.float32(127) / safe)), -127, 127).astype(np.float32)
    scale = np.where(amax > 0, amax / np.float32(127), np.float32(0)).astype(np.float32)
    return (codes * scale).astype(np.float64)


def full_forward(cfg, weights: dict, tokens, positions, kv_int8: bool = False) -> np.ndarray:
    """Logits fp64 [T][V] of a causal forward over all tokens at once, starting from an empty cache.
    kv_int8: k (after RoPE) and v pass through the 8-bit row compression instead of the bf16 rounding."""
    T = len(tokens)
    nq, nkv, d, F = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.ffn
    G = nq // nkv
    X = _bf16_bits_to_f64(weights["embed"][np.asarray(tokens)])               # [T][H]
    causal = np.tril(np.ones((T, T), bool))
    for lw in weights["layers"]:
        xn = _rms(X, _bf16_bits_to_f64(lw["input_norm"]), cfg.rms_eps)
        qkv = xn @ _bf16_bits_to_f64(lw["wqkv"]).T
        if lw["bqkv"] is not None:
            qkv = qkv + _bf16_bits_to_f64(lw["bqkv"])
        qkv = _f32(qkv)
        q = _rope_all(qkv[:, : nq * d].reshape(T, nq, d), positions, cfg.rope_theta)
        k = _rope_all(qkv[:, nq * d: (nq + nkv) * d].reshape(T, nkv, d), positions, cfg.rope_theta)
        v = qkv[:, (nq + nkv) * d:].reshape(T, nkv, d)
        k, v = (_int8_rows(k), _int8_rows(v)) if kv_int8 else (_round_bf16(k), _round_bf16(v))
        kq = np.repeat(k, G, axis=1)                                           # kv head h//G for q head h
        vq = np.repeat(v, G, axis=1)
        s = _f32(np.einsum("thd,shd->hts", q, kq) / np.sqrt(d))
        s = np.where(causal[None], s, -np.inf)
        p = np.exp(s - s.max(axis=-1, keepdims=True))
        p = _f32(p / p.sum(axis=-1, keepdims=True))
        o = _f32(np.einsum("hts,shd->thd", p, vq)).reshape(T, nq * d)
        X = _f32(X + _f32(o @ _bf16_bits_to_f64(lw["wo"]).T))
        xn = _rms(X, _bf16_bits_to_f64(lw["post_norm"]), cfg.rms_eps)
        gu = _f32(xn @ _bf16_bits_to_f64(lw["w_gate_up"]).T)
        a = _f32(gu[:, :F] / (1.0 + np.exp(-gu[:, :F])) * gu[:, F:])
        X = _f32(X + _f32(a @ _bf16_bits_to_f64(lw["w_down"]).T))
    xf = _rms(X, _bf16_bits_to_f64(weights["final_norm"]), cfg.rms_eps)
    return xf @ _bf16_bits_to_f64(weights["lm_head"]).T
