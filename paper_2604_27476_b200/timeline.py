"""Per-operator timeline of the persistent step kernel, from the device timestamps it records itself.

A context created while EDGEFM_PROFILE=1 is set makes thread 0 of every CTA store %globaltimer at fixed points of the
step (see edgefm_debug_profile in include/edgefm.h).  This module runs a few steps of a configuration and aggregates the
stamps of the last one:  `python bench.py --phase-timeline [--config NAME]` prints the table.
"""
from __future__ import annotations

import os

import numpy as np

STAMPS = ["qkv_staged", "qkv_done", "qkv_released", "att_done", "att_released", "o_staged", "o_done", "o_released",
          "gu_staged", "gu_done", "gu_released", "dn_staged", "dn_done", "dn_released"]


def collect(cfg, device="cuda:0", warm_steps=6, block_tokens=0):
    """Run warm_steps chained steps of cfg from its configured cache and return the stamp table of the last one,
    int64 [n_ctas][3 + 14 * n_layers] in nanoseconds.  block_tokens = 2: calls of edgefm_verify_block with two tokens
    (the proposal is arbitrary: an accepted and a rejected token cost the same)."""
    import torch
    from edgefm_synth import first_token, make_kv, make_weights
    from . import DecodeContext, edgefm_debug_profile, edgefm_sync_status, upload_weights

    old = os.environ.get("EDGEFM_PROFILE")
    os.environ["EDGEFM_PROFILE"] = "1"
    try:
        w = make_weights(cfg)
        k, v = make_kv(cfg)
        ptrs, keep = upload_weights(w, device)
        ctx = DecodeContext(cfg, ptrs, cfg.cache_len + max(block_tokens, 1) * warm_steps + 4, device, block_tokens=block_tokens)
    finally:
        if old is None:
            del os.environ["EDGEFM_PROFILE"]
        else:
            os.environ["EDGEFM_PROFILE"] = old
    from . import edgefm_debug_plan
    print("launch plan:", edgefm_debug_plan(ctx.handle))
    kd = torch.from_numpy(k.view(np.int16)).to(device)
    vd = torch.from_numpy(v.view(np.int16)).to(device)
    ctx.prefill_kv(kd, vd)
    if block_tokens > 1:
        ctx.verify_block([first_token(cfg)] + [5 % cfg.vocab] * (block_tokens - 1), cfg.first_position, want_logits=False)
        for _ in range(warm_steps - 1):
            ctx.verify_block([-1] + [7 % cfg.vocab] * (block_tokens - 1), -1, want_logits=False)
    else:
        ctx.step(first_token(cfg), cfg.first_position, want_logits=False, want_token=False)
        for _ in range(warm_steps - 1):
            ctx.step(-1, -1, want_logits=False, want_token=False)
    edgefm_sync_status(ctx.handle, torch.cuda.current_stream(torch.device(device)).cuda_stream)
    t = edgefm_debug_profile(ctx.handle).astype(np.int64)
    ctx.close()
    return t


def summarize(t, cfg) -> dict:
    """Durations in microseconds, mean over layers 1 .. L-1 (the first layer of a step starts cold)."""
    L = cfg.n_layers
    idx = lambda l, j: 1 + 14 * l + j
    prev = lambda l, j: idx(l, j - 1) if j > 0 else (idx(l - 1, 13) if l > 0 else 0)
    layers = range(1, L) if L > 1 else range(L)
    rows = {}
    for j, name in enumerate(STAMPS):
        mean_cta, max_cta = [], []
        for l in layers:
            a = t[:, idx(l, j)] - t[:, prev(l, j)]
            mean_cta.append(a.mean()); max_cta.append(a.max())
        rows[name] = (float(np.mean(mean_cta)) / 1e3, float(np.mean(max_cta)) / 1e3)
    per_layer = [(t[:, idx(l, 13)].max() - (t[:, idx(l - 1, 13)].max() if l > 0 else t[:, 0].min())) / 1e3 for l in range(L)]
    lm0 = t[:, idx(L - 1, 13)].max()
    out = {"rows": rows, "layer_us_first": float(per_layer[0]), "layer_us_mean": float(np.mean([per_layer[l] for l in layers])),
           "lm_staged_us": float((t[:, 1 + 14 * L].mean() - lm0) / 1e3), "lm_done_us": float((t[:, 1 + 14 * L + 1].max() - lm0) / 1e3),
           "step_us": float((t.max() - t[:, 0].min()) / 1e3)}
    return out


def format_table(s: dict, cfg) -> str:
    H, F, qd = cfg.hidden, cfg.ffn, cfg.n_q_heads * cfg.head_dim
    mb = {"qkv": cfg.qkv_rows * H * 2 / 1e6, "o": H * qd * 2 / 1e6, "gu": 2 * F * H * 2 / 1e6, "dn": F * H * 2 / 1e6}
    lines = [f"phase timeline of {cfg.name} (context {cfg.cache_len}); microseconds; mean over layers 1..L-1",
             f"{'stamp':14s} {'mean over CTAs':>15s} {'slowest CTA':>12s}"]
    for name in STAMPS:
        a, b = s["rows"][name]
        extra = ""
        key = name.split("_")[0]
        if name.endswith("_done") and key in mb:
            extra = f"   {mb[key]:7.2f} MB -> {mb[key] / b:6.2f} TB/s over the slowest CTA's phase" if b > 0 else ""
        lines.append(f"{name:14s} {a:15.2f} {b:12.2f}{extra}")
    lines.append(f"layer total: first {s['layer_us_first']:.2f}, others {s['layer_us_mean']:.2f}")
    lm_mb = cfg.vocab * H * 2 / 1e6
    lines.append(f"lm_head: staged {s['lm_staged_us']:.2f}, done {s['lm_done_us']:.2f}   {lm_mb:.1f} MB -> {lm_mb / max(s['lm_done_us'], 1e-9):.2f} TB/s")
    lines.append(f"whole step by these stamps: {s['step_us']:.1f}")
    return "\n".join(lines)
