"""ctypes access to oracle/edgefm_oracle.cpp (compiled on first use with g++)."""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SO = _HERE / "libedgefm_oracle.so"
_lib = None

_i64 = ctypes.c_int64
_p = ctypes.c_void_p


def build_oracle(force: bool = False) -> Path:
    src = _HERE / "edgefm_oracle.cpp"
    import hashlib
    stamp = _SO.with_suffix(".so.srchash")
    digest = hashlib.sha256(src.read_bytes()).hexdigest()
    if force or not _SO.exists() or not stamp.exists() or stamp.read_text().strip() != digest:
        tmp = _SO.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-fopenmp", "-o", str(tmp), str(src)])
        os.replace(tmp, _SO)
        stamp.write_text(digest + "\n")
    return _SO


def lib():
    global _lib
    if _lib is None:
        build_oracle()
        L = ctypes.CDLL(str(_SO))
        L.oracle_bf16_to_f32.restype = ctypes.c_float
        L.oracle_bf16_to_f32.argtypes = [ctypes.c_uint16]
        L.oracle_f32_to_bf16.restype = ctypes.c_uint16
        L.oracle_f32_to_bf16.argtypes = [ctypes.c_float]
        L.oracle_gemv.restype = None
        L.oracle_gemv.argtypes = [_p, _p, _p, _i64, _i64, _p]
        L.oracle_rmsnorm.restype = None
        L.oracle_rmsnorm.argtypes = [_p, _p, _i64, ctypes.c_double, _p]
        L.oracle_rope.restype = None
        L.oracle_rope.argtypes = [_p, _i64, _i64, ctypes.c_double]
        L.oracle_softmax.restype = None
        L.oracle_softmax.argtypes = [_p, _i64]
        L.oracle_silu.restype = ctypes.c_double
        L.oracle_silu.argtypes = [ctypes.c_double]
        L.oracle_argmax.restype = _i64
        L.oracle_argmax.argtypes = [_p, _i64]
        L.oracle_attention.restype = None
        L.oracle_attention.argtypes = [_p, _p, _p, _i64, _i64, _i64, _i64, _i64, _i64, _p]
        L.oracle_model_create.restype = _p
        L.oracle_model_create.argtypes = [_i64] * 7 + [ctypes.c_double, ctypes.c_double, _p, _p, _p, _p, _i64]
        L.oracle_model_destroy.restype = None
        L.oracle_model_destroy.argtypes = [_p]
        L.oracle_model_load_kv.restype = ctypes.c_int
        L.oracle_model_load_kv.argtypes = [_p, _p, _p, _i64]
        L.oracle_model_cur_len.restype = _i64
        L.oracle_model_cur_len.argtypes = [_p]
        L.oracle_model_export_kv.restype = None
        L.oracle_model_export_kv.argtypes = [_p, _p, _p]
        L.oracle_model_truncate.restype = ctypes.c_int
        L.oracle_model_truncate.argtypes = [_p, _i64]
        L.oracle_model_use_int8_kv.restype = ctypes.c_int
        L.oracle_model_use_int8_kv.argtypes = [_p]
        L.oracle_quantize_row.restype = None
        L.oracle_quantize_row.argtypes = [_p, _i64, _p, _p]
        L.oracle_attention_q8.restype = None
        L.oracle_attention_q8.argtypes = [_p, _p, _p, _p, _p, _i64, _i64, _i64, _i64, _p]
        L.oracle_model_export_kv_q8.restype = None
        L.oracle_model_export_kv_q8.argtypes = [_p, _p, _p, _p, _p]
        L.oracle_model_step.restype = _i64
        L.oracle_model_step.argtypes = [_p, _i64, _i64, _p]
        _lib = L
    return _lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


# ---- operator wrappers (numpy in, numpy out; bf16 operands are uint16 bit patterns) -------------
def gemv(W: np.ndarray, x: np.ndarray, bias: np.ndarray | None = None) -> np.ndarray:
    W = np.ascontiguousarray(W, np.uint16)
    x = _f32(x)
    rows, cols = W.shape
    assert x.shape == (cols,)
    y = np.empty(rows, np.float32)
    b = None if bias is None else np.ascontiguousarray(bias, np.uint16)
    lib().oracle_gemv(W.ctypes.data, x.ctypes.data, None if b is None else b.ctypes.data, rows, cols, y.ctypes.data)
    return y


def rmsnorm(x: np.ndarray, w: np.ndarray, eps: float) -> np.ndarray:
    x = _f32(x)
    w = np.ascontiguousarray(w, np.uint16)
    out = np.empty_like(x)
    lib().oracle_rmsnorm(x.ctypes.data, w.ctypes.data, x.size, eps, out.ctypes.data)
    return out


def rope(u: np.ndarray, pos: int, theta: float) -> np.ndarray:
    out = _f32(u).copy()
    lib().oracle_rope(out.ctypes.data, out.size, pos, theta)
    return out


def softmax(s: np.ndarray) -> np.ndarray:
    out = _f32(s).copy()
    lib().oracle_softmax(out.ctypes.data, out.size)
    return out


def silu(g: float) -> float:
    return float(lib().oracle_silu(g))


def argmax(v: np.ndarray) -> int:
    v = _f32(v)
    return int(lib().oracle_argmax(v.ctypes.data, v.size))


def restricted_greedy(logits: np.ndarray, token_ids) -> tuple[np.ndarray, int]:
    """Vocabulary pruning (named in the caption of Fig. 2, no algorithm given; reading: the greedy choice restricted
    to a subset of token ids, ascending).  -> (the subset's logits in subset order, the token id of the largest;
    equal maxima: the lowest id)."""
    ids = np.asarray(token_ids, np.int64)
    sub = _f32(logits)[ids]
    return sub, int(ids[argmax(sub)])


def f32_to_bf16(f: float) -> int:
    return int(lib().oracle_f32_to_bf16(f))


def bf16_to_f32(b: int) -> float:
    return float(lib().oracle_bf16_to_f32(b))


def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """q fp32 [n_q][d]; K, V uint16 (bf16) [n_kv][n][d] -> fp32 [n_q][d]."""
    q = _f32(q)
    K = np.ascontiguousarray(K, np.uint16)
    V = np.ascontiguousarray(V, np.uint16)
    n_q, d = q.shape
    n_kv, n, d2 = K.shape
    assert d2 == d and V.shape == K.shape
    out = np.empty_like(q)
    lib().oracle_attention(q.ctypes.data, K.ctypes.data, V.ctypes.data, n_q, n_kv, d, n, n * d, d, out.ctypes.data)
    return out


def quantize_row(x: np.ndarray) -> tuple[np.ndarray, float]:
    """Compression of one cache row (Sec. 3.9, C): fp32 [d] -> (int8 codes [d], fp32 scale)."""
    x = _f32(x)
    codes = np.empty(x.size, np.int8)
    scale = np.zeros(1, np.float32)
    lib().oracle_quantize_row(x.ctypes.data, x.size, codes.ctypes.data, scale.ctypes.data)
    return codes, float(scale[0])


def attention_q8(q: np.ndarray, K8: np.ndarray, Ks: np.ndarray, V8: np.ndarray, Vs: np.ndarray) -> np.ndarray:
    """q fp32 [n_q][d]; K8, V8 int8 [n_kv][n][d]; Ks, Vs fp32 [n_kv][n] -> fp32 [n_q][d]."""
    q = _f32(q)
    K8 = np.ascontiguousarray(K8, np.int8); V8 = np.ascontiguousarray(V8, np.int8)
    Ks = _f32(Ks); Vs = _f32(Vs)
    n_q, d = q.shape
    n_kv, n, d2 = K8.shape
    assert d2 == d and V8.shape == K8.shape and Ks.shape == (n_kv, n) and Vs.shape == (n_kv, n)
    out = np.empty_like(q)
    lib().oracle_attention_q8(q.ctypes.data, K8.ctypes.data, Ks.ctypes.data, V8.ctypes.data, Vs.ctypes.data, n_q, n_kv, d, n, out.ctypes.data)
    return out


class OracleModel:
    """Whole decoder with its own KV cache.  `weights` is the dict edgefm_synth.make_weights returns
    (or any dict of the same layout); the arrays are borrowed and kept alive here."""

    def __init__(self, cfg, weights: dict, max_context: int, kv_format: str = "bf16"):
        self.cfg = cfg
        self.kv_format = kv_format
        self._keep = weights
        ptrs = []
        for lw in weights["layers"]:
            for name in ("input_norm", "wqkv", "bqkv", "wo", "post_norm", "w_gate_up", "w_down"):
                a = lw[name]
                ptrs.append(None if a is None else a.ctypes.data)
        arr = (ctypes.c_void_p * len(ptrs))(*ptrs)
        self._h = lib().oracle_model_create(cfg.n_layers, cfg.hidden, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                                            cfg.ffn, cfg.vocab, cfg.rms_eps, cfg.rope_theta, arr,
                                            weights["embed"].ctypes.data, weights["final_norm"].ctypes.data,
                                            weights["lm_head"].ctypes.data, max_context)
        if not self._h:
            raise MemoryError("oracle_model_create failed")
        self.max_context = max_context
        if kv_format == "int8":
            if lib().oracle_model_use_int8_kv(self._h):
                raise RuntimeError("oracle_model_use_int8_kv failed")
        elif kv_format != "bf16":
            raise ValueError(kv_format)

    def load_kv(self, k: np.ndarray, v: np.ndarray) -> None:
        k = np.ascontiguousarray(k, np.uint16)
        v = np.ascontiguousarray(v, np.uint16)
        n = k.shape[2]
        if lib().oracle_model_load_kv(self._h, k.ctypes.data, v.ctypes.data, n):
            raise ValueError("too many positions")

    @property
    def cur_len(self) -> int:
        return int(lib().oracle_model_cur_len(self._h))

    def export_kv(self):
        c = self.cfg
        shape = (c.n_layers, c.n_kv_heads, self.max_context, c.head_dim)
        k = np.empty(shape, np.uint16)
        v = np.empty(shape, np.uint16)
        lib().oracle_model_export_kv(self._h, k.ctypes.data, v.ctypes.data)
        return k, v

    def truncate(self, n: int) -> None:
        if lib().oracle_model_truncate(self._h, n):
            raise ValueError("truncate beyond the cache length")

    def verify_block(self, tokens, pos: int):
        """Block verification as Sec. 3.11 states it, token by token: step every token of the block in turn (token t at
        position pos + t); proposal t + 1 is accepted if it equals the greedy token after token t, verification stops at the
        first rejection; the cache keeps the rows of the accepted tokens only.
        -> (logits fp32 [m][V] of all m tokens, n_accepted, next_token)."""
        start = self.cur_len
        logits, greedy = [], []
        for t, tok in enumerate(tokens):
            lg, nx = self.step(int(tok), pos + t)
            logits.append(lg); greedy.append(nx)
        n_acc = 1
        while n_acc < len(tokens) and int(tokens[n_acc]) == greedy[n_acc - 1]:
            n_acc += 1
        self.truncate(start + n_acc)
        return np.stack(logits), n_acc, greedy[n_acc - 1]

    def export_kv_q8(self):
        """-> (K codes int8, V codes int8 [L][n_kv][max_context][d], K scales fp32, V scales fp32 [L][n_kv][max_context])."""
        c = self.cfg
        shape = (c.n_layers, c.n_kv_heads, self.max_context, c.head_dim)
        k8 = np.empty(shape, np.int8); v8 = np.empty(shape, np.int8)
        ks = np.empty(shape[:3], np.float32); vs = np.empty(shape[:3], np.float32)
        lib().oracle_model_export_kv_q8(self._h, k8.ctypes.data, v8.ctypes.data, ks.ctypes.data, vs.ctypes.data)
        return k8, v8, ks, vs

    def step(self, token: int, pos: int):
        """-> (logits fp32[V], next_token)."""
        logits = np.empty(self.cfg.vocab, np.float32)
        nxt = int(lib().oracle_model_step(self._h, token, pos, logits.ctypes.data))
        if nxt < 0:
            raise RuntimeError("oracle step rejected (cache full or bad token)")
        return logits, nxt

    def close(self):
        if self._h:
            lib().oracle_model_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
