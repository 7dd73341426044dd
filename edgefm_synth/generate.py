"""Counter-based bf16 normal generator (C, OpenMP) and the per-tensor seeding recipe.

Weights come back as numpy uint16 arrays holding bf16 bit patterns, so that the very same host
buffers can be handed to the CPU oracle (by pointer) and uploaded to the GPU unchanged.
"""
from __future__ import annotations

import ctypes
import enum
import os
import subprocess
from pathlib import Path

import numpy as np

from .configs import DecoderConfig, GLOBAL_SEED

_HERE = Path(__file__).resolve().parent
_SO = _HERE / "libedgefm_synth.so"
_lib = None


def build_generator(force: bool = False) -> Path:
    src = _HERE / "gen.c"
    import hashlib
    stamp = _SO.with_suffix(".so.srchash")
    digest = hashlib.sha256(src.read_bytes()).hexdigest()
    if force or not _SO.exists() or not stamp.exists() or stamp.read_text().strip() != digest:
        tmp = _SO.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-o", str(tmp), str(src), "-lm"])
        os.replace(tmp, _SO)
        stamp.write_text(digest + "\n")
    return _SO


def _load():
    global _lib
    if _lib is None:
        build_generator()
        lib = ctypes.CDLL(str(_SO))
        lib.synth_u64.restype = ctypes.c_uint64
        lib.synth_u64.argtypes = [ctypes.c_uint64] * 3
        lib.synth_normal_bf16.restype = None
        lib.synth_normal_bf16.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64,
                                          ctypes.c_double, ctypes.c_void_p]
        _lib = lib
    return _lib


class TensorRole(enum.IntEnum):
    INPUT_NORM = 0
    WQKV = 1
    BQKV = 2
    WO = 3
    POST_NORM = 4
    W_GATE_UP = 5
    W_DOWN = 6
    K_CACHE = 7
    V_CACHE = 8
    # globals (layer index 0xFFFF)
    EMBED = 9
    FINAL_NORM = 10
    LM_HEAD = 11
    FIRST_TOKEN = 12


_GLOBAL_LAYER = 0xFFFF


def tensor_id(layer: int, role: TensorRole) -> int:
    return (layer << 8) | int(role)


def synth_u64(seed: int, tid: int, i: int) -> int:
    return int(_load().synth_u64(seed, tid, i))


def normal_bf16(seed: int, tid: int, shape, std: float, offset: int = 0) -> np.ndarray:
    """bf16 bit patterns (uint16) of N(0, std^2) samples for element indices offset .. offset+n-1."""
    out = np.empty(shape, dtype=np.uint16)
    _load().synth_normal_bf16(seed, tid, offset, out.size, float(std), out.ctypes.data)
    return out


def bf16_to_f32(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32)


_ONE_BF16 = 0x3F80


def make_weights(cfg: DecoderConfig, seed: int = GLOBAL_SEED) -> dict:
    """All weights of the decoder as uint16 (bf16 bits) numpy arrays.

    Matrices, embedding and biases ~ N(0, w_std); norm weights exactly 1.0.  Layouts:
      wqkv [(nq+2nkv)*d][H] (q heads, then k heads, then v heads), wo [H][nq*d],
      w_gate_up [2F][H] (gate rows then up rows), w_down [H][F], embed/lm_head [V][H].
    """
    H, F, V, R = cfg.hidden, cfg.ffn, cfg.vocab, cfg.qkv_rows
    qd = cfg.n_q_heads * cfg.head_dim
    layers = []
    for l in range(cfg.n_layers):
        lw = {
            "input_norm": np.full(H, _ONE_BF16, np.uint16),
            "wqkv": normal_bf16(seed, tensor_id(l, TensorRole.WQKV), (R, H), cfg.w_std),
            "bqkv": normal_bf16(seed, tensor_id(l, TensorRole.BQKV), (R,), cfg.w_std) if cfg.qkv_bias else None,
            "wo": normal_bf16(seed, tensor_id(l, TensorRole.WO), (H, qd), cfg.w_std),
            "post_norm": np.full(H, _ONE_BF16, np.uint16),
            "w_gate_up": normal_bf16(seed, tensor_id(l, TensorRole.W_GATE_UP), (2 * F, H), cfg.w_std),
            "w_down": normal_bf16(seed, tensor_id(l, TensorRole.W_DOWN), (H, F), cfg.w_std),
        }
        layers.append(lw)
    embed = normal_bf16(seed, tensor_id(_GLOBAL_LAYER, TensorRole.EMBED), (V, H), cfg.w_std)
    lm_head = embed if cfg.tied else normal_bf16(seed, tensor_id(_GLOBAL_LAYER, TensorRole.LM_HEAD), (V, H),
                                                 cfg.w_std)
    return {"layers": layers, "embed": embed, "final_norm": np.full(H, _ONE_BF16, np.uint16), "lm_head": lm_head}


def make_kv(cfg: DecoderConfig, seed: int = GLOBAL_SEED, n_positions: int | None = None):
    """K and V of the already-decoded prefix: uint16 (bf16) [L][n_kv][n_positions][d], ~N(0, kv_std)."""
    n = cfg.cache_len if n_positions is None else n_positions
    shape = (cfg.n_layers, cfg.n_kv_heads, n, cfg.head_dim)
    per_layer = shape[1] * shape[2] * shape[3]
    k = np.empty(shape, np.uint16)
    v = np.empty(shape, np.uint16)
    for l in range(cfg.n_layers):
        k[l] = normal_bf16(seed, tensor_id(l, TensorRole.K_CACHE), shape[1:], cfg.kv_std)
        v[l] = normal_bf16(seed, tensor_id(l, TensorRole.V_CACHE), shape[1:], cfg.kv_std)
    assert per_layer == k[0].size
    return k, v


def first_token(cfg: DecoderConfig, seed: int = GLOBAL_SEED) -> int:
    return synth_u64(seed, tensor_id(_GLOBAL_LAYER, TensorRole.FIRST_TOKEN), 0) % cfg.vocab
