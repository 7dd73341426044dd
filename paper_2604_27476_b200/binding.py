"""ctypes binding of include/edgefm.h: same names, argument marshalling only.

There is no fallback: if libedgefm.so is missing or cannot be loaded, load_library raises.
"""
from __future__ import annotations

import ctypes
import enum
from pathlib import Path

_PKG = Path(__file__).resolve().parent
_LIB_PATH = _PKG / "libedgefm.so"
_lib = None


class Status(enum.IntEnum):
    OK = 0
    ERR_INVALID_ARG = 1
    ERR_BAD_SHAPE = 2
    ERR_CONTEXT_FULL = 3
    ERR_OUT_OF_MEMORY = 4
    ERR_CUDA = 5
    ERR_TIMEOUT = 6


class EdgefmError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{Status(status).name}: {message}")
        self.status = Status(status)


class _Shape(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("hidden", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("ffn", ctypes.c_int32),
                ("vocab", ctypes.c_int32), ("rms_eps", ctypes.c_float), ("rope_theta", ctypes.c_float),
                ("qkv_bias", ctypes.c_int32)]


class _Options(ctypes.Structure):
    _fields_ = [("kv_format", ctypes.c_int32), ("block_tokens", ctypes.c_int32), ("reserved", ctypes.c_int32 * 6)]


class _LayerWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("input_norm", "wqkv", "bqkv", "wo", "post_norm", "w_gate_up", "w_down")]


class _Weights(ctypes.Structure):
    _fields_ = [("embed", ctypes.c_void_p), ("final_norm", ctypes.c_void_p), ("lm_head", ctypes.c_void_p),
                ("layers", ctypes.POINTER(_LayerWeights))]


EXPORTS = ("edgefm_create", "edgefm_prefill_kv", "edgefm_decode_step", "edgefm_destroy", "edgefm_get_length",
           "edgefm_export_kv", "edgefm_get_launches_per_step", "edgefm_last_error", "edgefm_version",
           "edgefm_sync_status", "edgefm_debug_profile", "edgefm_debug_set_wait_limit", "edgefm_debug_set_prefill_wait", "edgefm_debug_prefill_plan", "edgefm_debug_plan", "edgefm_debug_plan_operator", "edgefm_decode_step_static", "edgefm_set_vocab_subset",
           "edgefm_append_kv", "edgefm_create_with_options", "edgefm_export_kv_int8", "edgefm_verify_block", "edgefm_sync_length", "edgefm_prefill_tokens", "edgefm_prefill")


def library_path() -> Path:
    return _LIB_PATH


def load_library():
    global _lib
    if _lib is not None:
        return _lib
    path = _LIB_PATH
    if not path.exists():
        raise FileNotFoundError(f"{path} is missing: build it with `python -m paper_2604_27476_b200.build` "
                                "(there is no CPU fallback)")
    L = ctypes.CDLL(str(path))
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    L.edgefm_create.restype = ctypes.c_int
    L.edgefm_create.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Weights), i32, ctypes.POINTER(vp)]
    L.edgefm_create_with_options.restype = ctypes.c_int
    L.edgefm_create_with_options.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Weights), i32, ctypes.POINTER(_Options), ctypes.POINTER(vp)]
    L.edgefm_verify_block.restype = ctypes.c_int
    L.edgefm_verify_block.argtypes = [vp, ctypes.POINTER(i32), i32, i32, vp, vp, vp, vp]
    L.edgefm_prefill_tokens.restype = ctypes.c_int
    L.edgefm_prefill_tokens.argtypes = [vp, ctypes.POINTER(i32), i32, i32, vp]
    L.edgefm_prefill.restype = ctypes.c_int
    L.edgefm_prefill.argtypes = [vp, ctypes.POINTER(i32), i32, i32, vp, vp, vp]
    L.edgefm_sync_length.restype = ctypes.c_int
    L.edgefm_sync_length.argtypes = [vp, vp, ctypes.POINTER(i32)]
    L.edgefm_export_kv_int8.restype = ctypes.c_int
    L.edgefm_export_kv_int8.argtypes = [vp, vp, vp, vp, vp, vp]
    L.edgefm_prefill_kv.restype = ctypes.c_int
    L.edgefm_prefill_kv.argtypes = [vp, vp, vp, i32, i64, i64, i64, vp]
    L.edgefm_decode_step.restype = ctypes.c_int
    L.edgefm_decode_step.argtypes = [vp, i32, i32, vp, vp, vp]
    L.edgefm_destroy.restype = ctypes.c_int
    L.edgefm_destroy.argtypes = [vp]
    L.edgefm_get_length.restype = ctypes.c_int
    L.edgefm_get_length.argtypes = [vp, ctypes.POINTER(i32)]
    L.edgefm_export_kv.restype = ctypes.c_int
    L.edgefm_export_kv.argtypes = [vp, vp, vp, vp]
    L.edgefm_get_launches_per_step.restype = ctypes.c_int
    L.edgefm_get_launches_per_step.argtypes = [vp, ctypes.POINTER(i32)]
    L.edgefm_sync_status.restype = ctypes.c_int
    L.edgefm_sync_status.argtypes = [vp, vp]
    L.edgefm_debug_profile.restype = ctypes.c_int
    L.edgefm_debug_profile.argtypes = [vp, vp, i64, ctypes.POINTER(i32), ctypes.POINTER(i32)]
    L.edgefm_debug_set_wait_limit.restype = ctypes.c_int
    L.edgefm_debug_set_wait_limit.argtypes = [vp, ctypes.c_uint32, i32]
    L.edgefm_debug_set_prefill_wait.restype = ctypes.c_int
    L.edgefm_debug_set_prefill_wait.argtypes = [vp, ctypes.c_uint32, i32]
    L.edgefm_debug_plan.restype = ctypes.c_int
    L.edgefm_debug_plan.argtypes = [vp, ctypes.POINTER(i32)]
    L.edgefm_debug_plan_operator.restype = ctypes.c_int
    L.edgefm_debug_plan_operator.argtypes = [i32] * 8 + [vp, i64, vp, vp, i64, vp, vp, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    L.edgefm_decode_step_static.restype = ctypes.c_int
    L.edgefm_decode_step_static.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Weights), vp, vp, i32, i32, i32, i32, vp, vp, vp]
    L.edgefm_append_kv.restype = ctypes.c_int
    L.edgefm_append_kv.argtypes = [vp, vp, vp, i32, i32, i64, i64, i64, vp]
    L.edgefm_set_vocab_subset.restype = ctypes.c_int
    L.edgefm_set_vocab_subset.argtypes = [vp, vp, i32, vp]
    L.edgefm_last_error.restype = ctypes.c_char_p
    L.edgefm_last_error.argtypes = [vp]
    L.edgefm_version.restype = ctypes.c_char_p
    L.edgefm_version.argtypes = []
    _lib = L
    return L


def _check(status: int, ctx=None):
    if status != 0:
        raise EdgefmError(status, edgefm_last_error(ctx))


# ---- the C calls, one Python function each -------------------------------------------------------
def edgefm_version() -> str:
    return load_library().edgefm_version().decode()


def edgefm_last_error(ctx=None) -> str:
    return load_library().edgefm_last_error(ctx).decode()


KV_FORMATS = {"bf16": 0, "int8": 1}


def edgefm_create(shape: dict, weights: dict, max_context: int, kv_format: str | int | None = None, reserved=None, block_tokens: int = 0):
    """shape: dict with the fields of edgefm_shape; weights: {"embed", "final_norm", "lm_head": device
    pointers (int), "layers": [ {field: device pointer or None} ]}.  Returns the opaque context handle.
    kv_format: None = edgefm_create; "bf16" / "int8" (or the raw integer) = edgefm_create_with_options."""
    L = load_library()
    sh = _Shape(**shape)
    layers = weights["layers"]
    arr = (_LayerWeights * max(1, len(layers)))()
    for i, lw in enumerate(layers):
        for name, _ in _LayerWeights._fields_:
            setattr(arr[i], name, lw.get(name))
    w = _Weights(weights["embed"], weights["final_norm"], weights["lm_head"], arr)
    out = ctypes.c_void_p()
    if kv_format is None and not block_tokens and not reserved:
        _check(L.edgefm_create(ctypes.byref(sh), ctypes.byref(w), max_context, ctypes.byref(out)))
    else:
        fmt = 0 if kv_format is None else (KV_FORMATS.get(kv_format, kv_format) if isinstance(kv_format, str) else int(kv_format))
        opt = _Options(fmt, int(block_tokens), (ctypes.c_int32 * 6)(*(list(reserved or [])[:6] + [0] * 6)[:6]))
        _check(L.edgefm_create_with_options(ctypes.byref(sh), ctypes.byref(w), max_context, ctypes.byref(opt), ctypes.byref(out)))
    return out


def edgefm_prefill_kv(ctx, k_ptr, v_ptr, n_positions, stride_layer, stride_head, stride_pos, stream=None):
    _check(load_library().edgefm_prefill_kv(ctx, k_ptr, v_ptr, n_positions, stride_layer, stride_head, stride_pos, stream), ctx)


def edgefm_decode_step(ctx, token_id, position, stream=None, logits_out=None, next_token_out=None):
    _check(load_library().edgefm_decode_step(ctx, token_id, position, stream, logits_out, next_token_out), ctx)


def edgefm_destroy(ctx):
    _check(load_library().edgefm_destroy(ctx))


def edgefm_get_length(ctx) -> int:
    n = ctypes.c_int32()
    _check(load_library().edgefm_get_length(ctx, ctypes.byref(n)), ctx)
    return n.value


def edgefm_get_launches_per_step(ctx) -> int:
    n = ctypes.c_int32()
    _check(load_library().edgefm_get_launches_per_step(ctx, ctypes.byref(n)), ctx)
    return n.value


def _marshal_weights(weights: dict):
    layers = weights["layers"]
    arr = (_LayerWeights * max(1, len(layers)))()
    for i, lw in enumerate(layers):
        for name, _ in _LayerWeights._fields_:
            setattr(arr[i], name, lw.get(name))
    return _Weights(weights["embed"], weights["final_norm"], weights["lm_head"], arr), arr


def edgefm_decode_step_static(shape: dict, weights: dict, k_cache_ptr, v_cache_ptr, max_context, cur_len, token_id, position,
                              stream=None, logits_out=None, next_token_out=None):
    """One decode step with no allocation anywhere: work buffers come from the library's fixed scratch array, the
    KV cache ([L][n_kv][max_context][d] bf16, device) and the cache length are the caller's."""
    sh = _Shape(**shape)
    w, keep = _marshal_weights(weights)
    _check(load_library().edgefm_decode_step_static(ctypes.byref(sh), ctypes.byref(w), k_cache_ptr, v_cache_ptr, max_context,
                                                    cur_len, token_id, position, stream, logits_out, next_token_out))


def edgefm_append_kv(ctx, k_ptr, v_ptr, start, n_positions, stride_layer, stride_head, stride_pos, stream=None):
    _check(load_library().edgefm_append_kv(ctx, k_ptr, v_ptr, start, n_positions, stride_layer, stride_head, stride_pos, stream), ctx)


def edgefm_set_vocab_subset(ctx, token_ids, stream=None):
    """token_ids: strictly ascending int32 ids (any sequence or numpy array) the greedy choice is restricted to;
    None or empty restores the full vocabulary."""
    import numpy as np
    ids = np.ascontiguousarray(np.asarray([] if token_ids is None else token_ids, dtype=np.int32))
    _check(load_library().edgefm_set_vocab_subset(ctx, ids.ctypes.data if ids.size else None, int(ids.size), stream), ctx)


def edgefm_sync_status(ctx, stream=None):
    _check(load_library().edgefm_sync_status(ctx, stream), ctx)


def edgefm_debug_prefill_plan(epilogue, M, N, K, num_sms=148):
    """(wide, splits) the prefill planner gives a contraction (host only)."""
    L = load_library()
    L.edgefm_debug_prefill_plan.restype = ctypes.c_int
    L.edgefm_debug_prefill_plan.argtypes = [ctypes.c_int32] * 5 + [ctypes.POINTER(ctypes.c_int32)]
    out = (ctypes.c_int32 * 2)()
    _check(L.edgefm_debug_prefill_plan(epilogue, M, N, K, num_sms, out), None)
    return int(out[0]), int(out[1])


def edgefm_debug_set_prefill_wait(ctx, polls, extra_arrivals=0):
    _check(load_library().edgefm_debug_set_prefill_wait(ctx, polls, extra_arrivals), ctx)


def edgefm_debug_set_wait_limit(ctx, limit_ns, extra_barrier_arrivals=0):
    _check(load_library().edgefm_debug_set_wait_limit(ctx, limit_ns, extra_barrier_arrivals), ctx)


def edgefm_debug_plan(ctx) -> dict:
    """Launch geometry of the context's step kernel."""
    out = (ctypes.c_int32 * 8)()
    _check(load_library().edgefm_debug_plan(ctx, out), ctx)
    keys = ("ctas", "consumer_warps", "ring_slots_per_warp", "slot_bytes", "dynamic_smem_bytes", "max_tiles_per_cta", "schedule_smem_bytes",
            "long_context_build")
    return dict(zip(keys, list(out)))


def edgefm_debug_plan_operator(kind, units, K, head_half, op_index, n_ctas, n_warps, slot_rows):
    """Host-only: the tile schedule the planner makes for one operator.  Returns a dict with
    tiles [cta][warp] -> list of decoded tile dicts, combines [cta] -> list of dicts, variant_rows."""
    import numpy as np
    L = load_library()
    per_warp = np.zeros(n_ctas * n_warps, np.int32)
    per_cta = np.zeros(n_ctas, np.int32)
    variants = np.zeros(4, np.int32)
    nt, nc = ctypes.c_int64(), ctypes.c_int64()
    args = (kind, units, K, head_half, op_index, n_ctas, n_warps, slot_rows)
    _check(L.edgefm_debug_plan_operator(*args, None, 0, per_warp.ctypes.data, None, 0, per_cta.ctypes.data, variants.ctypes.data,
                                        ctypes.byref(nt), ctypes.byref(nc)))
    tiles = np.zeros(max(nt.value, 1), np.uint64)
    comb = np.zeros(max(nc.value, 1) * 4, np.uint32)
    _check(L.edgefm_debug_plan_operator(*args, tiles.ctypes.data, tiles.size, per_warp.ctypes.data, comb.ctypes.data, nc.value, per_cta.ctypes.data,
                                        variants.ctypes.data, ctypes.byref(nt), ctypes.byref(nc)))
    out_tiles, pos = [], 0
    for c in range(n_ctas):
        row = []
        for w in range(n_warps):
            lst = []
            for _ in range(per_warp[c * n_warps + w]):
                d = int(tiles[pos]); pos += 1
                x, y = d & 0xffffffff, d >> 32
                lst.append(dict(unit_base=x & 0xfffff, kcol=(x >> 20) & 0xff, variant=(x >> 28) & 3, first=bool(x >> 30 & 1), flush=bool(x >> 31 & 1),
                                m=y & 31, v0=(y >> 5) & 15, direct=bool(y >> 9 & 1), slot=(y >> 10) & 1023, op=(y >> 20) & 7))
            row.append(lst)
        out_tiles.append(row)
    out_comb, pos = [], 0
    for c in range(n_ctas):
        lst = []
        for _ in range(per_cta[c]):
            e = comb[4 * pos: 4 * pos + 4]; pos += 1
            lst.append(dict(unit_base=int(e[0]), m=int(e[1]) & 0xff, v0=int(e[1]) >> 8, first_slot=int(e[2]), n_slots=int(e[3])))
        out_comb.append(lst)
    return dict(tiles=out_tiles, combines=out_comb, variant_rows=[int(v) for v in variants if v])


def edgefm_debug_profile(ctx):
    """-> numpy uint64 [n_ctas][stride] of device timestamps (ns) of the last step, or None when profiling is off."""
    import numpy as np
    L = load_library()
    n, st = ctypes.c_int32(), ctypes.c_int32()
    _check(L.edgefm_debug_profile(ctx, None, 0, ctypes.byref(n), ctypes.byref(st)), ctx)
    if n.value == 0:
        return None
    out = np.zeros((n.value, st.value), np.uint64)
    _check(L.edgefm_debug_profile(ctx, out.ctypes.data, out.size, ctypes.byref(n), ctypes.byref(st)), ctx)
    return out


def edgefm_export_kv(ctx, k_out_ptr, v_out_ptr, stream=None):
    _check(load_library().edgefm_export_kv(ctx, k_out_ptr, v_out_ptr, stream), ctx)


def edgefm_verify_block(ctx, tokens, position, stream=None, logits_out=None, n_accepted_out=None, next_token_out=None):
    arr = (ctypes.c_int32 * max(1, len(tokens)))(*[int(t) for t in tokens])
    _check(load_library().edgefm_verify_block(ctx, arr, len(tokens), position, stream, logits_out, n_accepted_out, next_token_out), ctx)


def edgefm_prefill_tokens(ctx, tokens, position, stream=None):
    arr = (ctypes.c_int32 * max(1, len(tokens)))(*[int(t) for t in tokens])
    _check(load_library().edgefm_prefill_tokens(ctx, arr, len(tokens), position, stream), ctx)


def edgefm_prefill(ctx, tokens, position, stream=None, logits_out=None, next_token_out=None):
    arr = (ctypes.c_int32 * max(1, len(tokens)))(*[int(t) for t in tokens])
    _check(load_library().edgefm_prefill(ctx, arr, len(tokens), position, stream, logits_out, next_token_out), ctx)


def edgefm_sync_length(ctx, stream=None) -> int:
    n = ctypes.c_int32()
    _check(load_library().edgefm_sync_length(ctx, stream, ctypes.byref(n)), ctx)
    return n.value


def edgefm_export_kv_int8(ctx, k_codes_ptr, v_codes_ptr, k_scales_ptr, v_scales_ptr, stream=None):
    _check(load_library().edgefm_export_kv_int8(ctx, k_codes_ptr, v_codes_ptr, k_scales_ptr, v_scales_ptr, stream), ctx)


# ---- convenience for tests and the benchmark: torch owns the device memory ------------------------
def upload_weights(host_weights: dict, device="cuda:0"):
    """Copy a dict of numpy uint16 (bf16 bits) arrays (layout of edgefm_weights) to the device.
    Returns (pointer dict for edgefm_create, list of torch tensors that must be kept alive)."""
    import numpy as np
    import torch

    keep = []

    def up(a):
        if a is None:
            return None
        t = torch.from_numpy(a.view(np.int16)).to(device)
        keep.append(t)
        return t.data_ptr()

    embed = up(host_weights["embed"])
    lm = embed if host_weights["lm_head"] is host_weights["embed"] else up(host_weights["lm_head"])
    ptrs = {"embed": embed, "final_norm": up(host_weights["final_norm"]), "lm_head": lm,
            "layers": [{k: up(v) for k, v in lw.items()} for lw in host_weights["layers"]]}
    return ptrs, keep


class DecodeContext:
    """RAII wrapper of one edgefm context with torch-allocated I/O buffers."""

    def __init__(self, cfg, device_weight_ptrs: dict, max_context: int, device="cuda:0", kv_format: str | None = None, block_tokens: int = 0):
        import torch

        self.cfg = cfg
        self.kv_format = kv_format or "bf16"
        self.device = torch.device(device)
        self.max_context = max_context
        shape = dict(n_layers=cfg.n_layers, hidden=cfg.hidden, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                     head_dim=cfg.head_dim, ffn=cfg.ffn, vocab=cfg.vocab, rms_eps=cfg.rms_eps,
                     rope_theta=cfg.rope_theta, qkv_bias=int(cfg.qkv_bias))
        with torch.cuda.device(self.device):
            self.handle = edgefm_create(shape, device_weight_ptrs, max_context, kv_format, block_tokens=block_tokens)
        self.block_tokens = max(1, block_tokens)
        # rows for the longest block a call may carry: block_tokens through the step kernel, up to 8 through the dense path
        self.block_logits = torch.empty((max(self.block_tokens, 8), cfg.vocab), dtype=torch.float32, device=self.device)
        self.logits = self.block_logits[0]
        self.next_token = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.n_accepted = torch.zeros(1, dtype=torch.int32, device=self.device)

    def _stream(self):
        import torch
        return torch.cuda.current_stream(self.device).cuda_stream

    def prefill_kv(self, k, v):
        """k, v: torch int16/bf16 tensors [L][n_kv][n][d] on the device (any strides with contiguous last dim)."""
        n = k.shape[2]
        assert k.stride() == v.stride() and k.stride(3) == 1
        edgefm_prefill_kv(self.handle, k.data_ptr(), v.data_ptr(), n, k.stride(0), k.stride(1), k.stride(2), self._stream())

    def append_kv(self, start, k=None, v=None):
        """Keep the first `start` slots, then append k, v ([L][n_kv][n][d], device) behind them; k = None only truncates."""
        if k is None:
            edgefm_append_kv(self.handle, None, None, start, 0, 0, 0, 0, self._stream())
            return
        assert k.stride() == v.stride() and k.stride(3) == 1
        edgefm_append_kv(self.handle, k.data_ptr(), v.data_ptr(), start, k.shape[2], k.stride(0), k.stride(1), k.stride(2), self._stream())

    def reset(self):
        """Empty the cache (cache length 0)."""
        edgefm_prefill_kv(self.handle, None, None, 0, 0, 0, 0, self._stream())

    def step(self, token_id=-1, position=-1, want_logits=True, want_token=True):
        edgefm_decode_step(self.handle, token_id, position, self._stream(),
                           self.logits.data_ptr() if want_logits else None,
                           self.next_token.data_ptr() if want_token else None)

    def verify_block(self, tokens, position=-1, want_logits=True):
        """One call for a block of tokens (tokens[0] may be -1); results in block_logits[:m], n_accepted, next_token."""
        edgefm_verify_block(self.handle, tokens, position, self._stream(), self.block_logits.data_ptr() if want_logits else None,
                            self.n_accepted.data_ptr(), self.next_token.data_ptr())

    def prefill_tokens(self, tokens, position):
        """Append the cache rows of the given tokens (computed from the weights); the greedy next token stays on the device."""
        edgefm_prefill_tokens(self.handle, tokens, position, self._stream())

    def prefill(self, tokens, position=0, want_logits=True):
        """The prefill phase for a prompt: dense contractions for all but the last token, a decode step for the last."""
        edgefm_prefill(self.handle, tokens, position, self._stream(), self.logits.data_ptr() if want_logits else None,
                       self.next_token.data_ptr())

    def sync_status(self):
        """Synchronise the stream and raise EdgefmError(ERR_TIMEOUT) if a bounded device-side wait ran out."""
        edgefm_sync_status(self.handle, self._stream())

    def sync_length(self) -> int:
        return edgefm_sync_length(self.handle, self._stream())

    def set_vocab_subset(self, token_ids):
        """Restrict the output layer to these token ids (ascending); None restores the full vocabulary.  With a subset
        of n ids, logits[:n] holds the subset's logits in subset order."""
        edgefm_set_vocab_subset(self.handle, token_ids, self._stream())

    def export_kv(self):
        import torch
        c = self.cfg
        shape = (c.n_layers, c.n_kv_heads, self.max_context, c.head_dim)
        k = torch.empty(shape, dtype=torch.int16, device=self.device)
        v = torch.empty(shape, dtype=torch.int16, device=self.device)
        edgefm_export_kv(self.handle, k.data_ptr(), v.data_ptr(), self._stream())
        return k, v

    def export_kv_int8(self):
        """Compressed cache: (K codes, V codes int8 [L][n_kv][max_context][d], K scales, V scales fp32 [L][n_kv][max_context])."""
        import torch
        c = self.cfg
        shape = (c.n_layers, c.n_kv_heads, self.max_context, c.head_dim)
        k8 = torch.empty(shape, dtype=torch.int8, device=self.device)
        v8 = torch.empty(shape, dtype=torch.int8, device=self.device)
        ks = torch.empty(shape[:3], dtype=torch.float32, device=self.device)
        vs = torch.empty(shape[:3], dtype=torch.float32, device=self.device)
        edgefm_export_kv_int8(self.handle, k8.data_ptr(), v8.data_ptr(), ks.data_ptr(), vs.data_ptr(), self._stream())
        return k8, v8, ks, vs

    @property
    def cur_len(self) -> int:
        return edgefm_get_length(self.handle)

    @property
    def launches_per_step(self) -> int:
        return edgefm_get_launches_per_step(self.handle)

    def close(self):
        if getattr(self, "handle", None):
            edgefm_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
