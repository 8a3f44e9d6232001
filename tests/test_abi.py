"""CPU-side checks of the C-ABI boundary: the library loads, exports every declared symbol, and
rejects bad arguments on the host before anything touches a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2604_06832_b200 import binding as B
from paper_2604_06832_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return B.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "fdvlm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fdvlm_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    syms = declared_symbols()
    assert len(syms) >= 18
    for s in syms:
        assert hasattr(lib, s), f"{s} declared in fdvlm.h but not exported"
        assert s in B.EXPORTS, f"{s} has no ctypes prototype"
    assert set(B.EXPORTS) == set(syms)
    assert b"sm_100a" in lib.fdvlm_version()


def good_cfg(**kw):
    d = dict(n_layers=1, hidden=64, n_q_heads=2, n_kv_heads=1, head_dim=64, intermediate=128, vocab=100, mask_id=99,
             rms_eps=1e-6, rope_theta=1e6, tie_embeddings=1, dtype=B.DT_F32, max_seq=64, max_block=8, kv_dtype=B.KV_BF16)
    d.update(kw)
    return B.Config(*[d[n] for n, _ in B.Config._fields_])


def fake_weights(n_layers=1, lm_head=None):
    layers = (B.LayerWeights * n_layers)()
    for lw in layers:
        for name in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "g_attn", "g_mlp"):
            setattr(lw, name, 0x1000)
    return B.Weights(0x1000, lm_head, None, 0x1000, layers), layers


@pytest.mark.parametrize("kw,code", [
    (dict(head_dim=48), B.ERR_UNSUPPORTED),
    (dict(n_q_heads=3, n_kv_heads=2), B.ERR_INVALID_ARG),
    (dict(max_block=65), B.ERR_INVALID_ARG),
    (dict(max_block=0), B.ERR_INVALID_ARG),
    (dict(mask_id=100), B.ERR_INVALID_ARG),
    (dict(dtype=7), B.ERR_INVALID_ARG),
    (dict(hidden=60), B.ERR_UNSUPPORTED),
    (dict(dtype=B.DT_BF16, hidden=72), B.ERR_UNSUPPORTED),
    (dict(max_seq=4), B.ERR_INVALID_ARG),
    (dict(rms_eps=0.0), B.ERR_INVALID_ARG),
    (dict(n_layers=0), B.ERR_INVALID_ARG),
    (dict(kv_dtype=2), B.ERR_INVALID_ARG),
])
def test_create_rejects_bad_config_before_touching_the_device(lib, kw, code):
    w, _keep = fake_weights()
    out = C.c_void_p()
    assert lib.fdvlm_create(C.byref(good_cfg(**kw)), C.byref(w), None, C.byref(out)) == code
    assert out.value is None and lib.fdvlm_last_error(None) != b""


def test_create_rejects_bad_weight_sets(lib):
    out = C.c_void_p()
    w, _k = fake_weights(lm_head=0x1000)                      # tied but lm_head given
    assert lib.fdvlm_create(C.byref(good_cfg()), C.byref(w), None, C.byref(out)) == B.ERR_INVALID_ARG
    w, _k = fake_weights()                                    # untied but lm_head missing
    assert lib.fdvlm_create(C.byref(good_cfg(tie_embeddings=0)), C.byref(w), None, C.byref(out)) == B.ERR_INVALID_ARG
    w, layers = fake_weights()
    layers[0].w_up = None
    assert lib.fdvlm_create(C.byref(good_cfg()), C.byref(w), None, C.byref(out)) == B.ERR_INVALID_ARG
    w, layers = fake_weights()
    layers[0].bq = 0x1000                                     # one bias only
    assert lib.fdvlm_create(C.byref(good_cfg()), C.byref(w), None, C.byref(out)) == B.ERR_INVALID_ARG
    w, layers = fake_weights()                                # fp8 without scales
    assert lib.fdvlm_create(C.byref(good_cfg(dtype=B.DT_FP8)), C.byref(w), None, C.byref(out)) == B.ERR_INVALID_ARG
    assert lib.fdvlm_create(None, C.byref(w), None, C.byref(out)) == B.ERR_INVALID_ARG


def test_null_handle_calls_do_not_crash(lib):
    assert lib.fdvlm_cache_len(None) == B.ERR_INVALID_ARG
    assert lib.fdvlm_reset(None) == B.ERR_INVALID_ARG
    assert lib.fdvlm_commit_block(None, None) == B.ERR_INVALID_ARG
    assert lib.fdvlm_prefill(None, None, 0, None, 0, None) == B.ERR_INVALID_ARG
    assert lib.fdvlm_synchronize(None) == B.ERR_INVALID_ARG
    assert lib.fdvlm_debug_poison(None, 1) == B.ERR_INVALID_ARG
    assert lib.fdvlm_decode_block(None, 4, None, None, None, None) == B.ERR_INVALID_ARG
    assert lib.fdvlm_profile_read_chain(None, None, 0, None) == B.ERR_INVALID_ARG
    lib.fdvlm_destroy(None)


def test_op_argument_checks(lib):
    assert lib.fdvlm_op_linear(None, None, None, None, None, 1, 1, 8, B.DT_F32, None, None) == B.ERR_INVALID_ARG
    assert lib.fdvlm_op_linear(0x10, 0x10, None, None, 0x10, 65, 8, 8, B.DT_F32, 0x10, None) == B.ERR_INVALID_ARG
    assert lib.fdvlm_op_linear(0x10, 0x10, None, None, 0x10, 4, 8, 12, B.DT_F32, 0x10, None) == B.ERR_INVALID_ARG
    assert lib.fdvlm_op_linear(0x10, 0x10, None, None, 0x10, 4, 8, 16, B.DT_FP8, 0x10, None) == B.ERR_INVALID_ARG
    assert lib.fdvlm_op_linear(0x10, 0x10, None, None, 0x10, 4, 8, 16, B.DT_BF16, None, None) == B.ERR_INVALID_ARG   # no workspace
    assert lib.fdvlm_op_attention(0x10, 0x10, 0x10, 0x10, 4, 60, 62, 4, 2, 64, 0, B.DT_F32, B.KV_BF16, None, None) == B.ERR_INVALID_ARG
    assert lib.fdvlm_op_attention(0x10, 0x10, 0x10, 0x10, 4, 0, 62, 4, 3, 64, 0, B.DT_F32, B.KV_BF16, None, None) == B.ERR_INVALID_ARG
    assert lib.fdvlm_op_attention(0x10, 0x10, 0x10, 0x10, 4, 0, 62, 4, 2, 64, 0, B.DT_BF16, 5, 0x10, None) == B.ERR_INVALID_ARG
    # every workspace starts with the kernels' status words, so it is never empty
    assert lib.fdvlm_op_linear_workspace_bytes(32, 2048, 2048, B.DT_BF16) >= 256
    # (with a GPU present the fp8 figure also holds the f16 copy of the rows; without one both are the CUDA-core sizes)
    assert (lib.fdvlm_op_linear_workspace_bytes(32, 2048, 2048, B.DT_FP8)
            >= lib.fdvlm_op_linear_workspace_bytes(32, 2048, 2048, B.DT_BF16))


def test_no_gpu_means_loud_failure_not_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    w, _k = fake_weights()
    out = C.c_void_p()
    assert lib.fdvlm_create(C.byref(good_cfg()), C.byref(w), None, C.byref(out)) == B.ERR_CUDA
    assert b"CUDA" in lib.fdvlm_last_error(None) or b"device" in lib.fdvlm_last_error(None)
