"""Diagnostics of the library on a GPU: the in-kernel timestamps, the status query, and a second context on the
same weights."""
import os
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest

from edgefm_synth import CONFIGS, first_token
from helpers import Pair, assert_logits_close

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parents[1]


def _run_child(code: str, env_extra: dict) -> str:
    env = dict(os.environ, **env_extra)
    out = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stdout + out.stderr
    return out.stdout


CHILD = r'''
import sys, numpy as np, torch
sys.path.insert(0, "tests")
from edgefm_synth import CONFIGS, first_token
from helpers import Pair, assert_logits_close
from paper_2604_27476_b200 import edgefm_debug_profile, edgefm_sync_status
cfg = CONFIGS["tiny"].with_(qkv_bias=True)
pair = Pair(cfg, cache_len=200, max_context=260)
tok, pos = first_token(cfg), 200
worst = 0.0
for s in range(40):
    ref, nxt = pair.oracle.step(tok, pos)
    pair.ctx.step(tok, pos)
    torch.cuda.synchronize()
    ma, rl = assert_logits_close(pair.ctx.logits.cpu().numpy(), ref, f"step {s}")
    worst = max(worst, ma)
    tok, pos = nxt, pos + 1
edgefm_sync_status(pair.ctx.handle, torch.cuda.current_stream().cuda_stream)
prof = edgefm_debug_profile(pair.ctx.handle)
print("LAUNCHES", pair.ctx.launches_per_step, "WORST", worst, "PROF", None if prof is None else prof.shape,
      None if prof is None else bool((np.diff(prof[:, :3 + 14 * cfg.n_layers].astype(np.int64), axis=1) >= 0).all()))
pair.close()
'''


def test_persistent_kernel_with_timestamps_matches_oracle_and_timestamps_are_ordered():
    out = _run_child(CHILD, {"EDGEFM_PROFILE": "1"})
    assert "LAUNCHES 1 " in out
    assert "PROF (" in out and ", 31) True" in out       # [CTAs][3 + 14 * layers] stamps, non-decreasing per CTA


def test_two_contexts_share_weights_and_do_not_interfere():
    import torch
    from paper_2604_27476_b200 import DecodeContext
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, cache_len=50, max_context=60)
    try:
        other = DecodeContext(cfg, pair.ptrs, 60)
        other.prefill_kv(pair.kd, pair.vd)
        tok, pos = first_token(cfg), 50
        for s in range(3):                              # interleaved steps on one stream
            pair.ctx.step(tok + s, pos + s)
            other.step(tok + s, pos + s)
        torch.cuda.synchronize()
        assert torch.equal(pair.ctx.logits, other.logits) and torch.equal(pair.ctx.next_token, other.next_token)
        ka, va = pair.ctx.export_kv(); kb, vb = other.export_kv()
        assert torch.equal(ka, kb) and torch.equal(va, vb)
        other.close()
    finally:
        pair.close()
