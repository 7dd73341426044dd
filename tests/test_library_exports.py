"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parents[1]


def declared_symbols():
    text = (ROOT / "include" / "edgefm.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(edgefm_[a-z_]+)\s*\(", text)))


def test_library_loads_and_exports_every_declared_symbol():
    from paper_2604_27476_b200 import build as B, binding
    B.build()
    lib = binding.load_library()
    names = declared_symbols()
    assert {"edgefm_create", "edgefm_prefill_kv", "edgefm_decode_step", "edgefm_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) >= set(n for n in names if n != "edgefm_ctx")
    assert "sm_100a" in binding.edgefm_version()


def test_host_side_validation_runs_without_a_gpu():
    import torch
    from paper_2604_27476_b200 import EdgefmError, Status, edgefm_create, load_library
    shape = dict(n_layers=1, hidden=64, n_q_heads=1, n_kv_heads=1, head_dim=64, ffn=64, vocab=10, rms_eps=1e-6,
                 rope_theta=1e6, qkv_bias=0)
    lw = dict(input_norm=256, wqkv=256, bqkv=None, wo=256, post_norm=256, w_gate_up=256, w_down=256)
    w = dict(embed=256, final_norm=256, lm_head=256, layers=[lw])
    with pytest.raises(EdgefmError) as ei:
        edgefm_create(dict(shape, head_dim=80), w, 8)
    assert ei.value.status == Status.ERR_BAD_SHAPE
    with pytest.raises(EdgefmError) as ei:
        edgefm_create(shape, w, -1)
    assert ei.value.status == Status.ERR_INVALID_ARG
    if not torch.cuda.is_available():
        with pytest.raises(EdgefmError) as ei:                 # no CPU fallback: fails loudly
            edgefm_create(shape, w, 8)
        assert ei.value.status == Status.ERR_CUDA
    L = load_library()
    assert L.edgefm_destroy(None) == 0
    assert L.edgefm_decode_step(None, 0, 0, None, None, None) == int(Status.ERR_INVALID_ARG)
