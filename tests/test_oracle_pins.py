"""Pins for the CPU oracle: everything here is fixed by the paper or by mathematics, not by the
oracle's own formulas (closed forms, invariants, brute force, textbook reductions, and an
independent torch restatement)."""
import math

import numpy as np
import pytest
import torch

from oracle import fdvlm_oracle as orc
from paper_2604_06832_b200 import inputs as I

MICRO = I.ModelShape(n_layers=2, hidden=32, n_q_heads=4, n_kv_heads=2, head_dim=8, intermediate=48,
                     vocab=64, mask_id=63, tie_embeddings=True, dtype=I.F32)


def make(shape=MICRO, seed=3, std=0.3, **kw):
    w = I.make_weights(shape, seed, std=std, **kw)
    return orc.Oracle(shape, I.weights_to_numpy(w)), w


def prefix(shape, ne, nt, seed=7):
    e, t = I.make_prefix(shape, ne, nt, seed)
    return I.as_numpy_storage(e), t.numpy()


# ---- storage decoding -----------------------------------------------------------------------
def test_decode_bf16_matches_torch_cast():
    bits = np.arange(0, 65536, dtype=np.uint16)
    ref = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    got = orc.decode_bf16(bits)
    ok = np.isfinite(ref)
    assert np.array_equal(got[ok], ref[ok])


def test_decode_e4m3_format_facts():
    # values fixed by the OCP FP8 E4M3 definition
    t = orc.decode_e4m3(np.arange(256, dtype=np.uint8))
    assert t[0] == 0.0 and t[0x38] == 1.0 and t[0x7E] == 448.0 and t[0xFE] == -448.0
    assert t[0x01] == 2.0 ** -9 and t[0x08] == 2.0 ** -6 and math.isnan(t[0x7F]) and math.isnan(t[0xFF])
    ref = torch.arange(256, dtype=torch.int16).to(torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    ok = np.isfinite(ref)
    assert np.array_equal(t[ok], ref[ok])


# ---- P9: closed forms -----------------------------------------------------------------------
def test_rmsnorm_constant_row_closed_form():
    c, eps = 3.0, 1e-6
    g = np.linspace(0.5, 2.0, 16)
    out = orc.rmsnorm(np.full((1, 16), c), g, eps)
    assert np.allclose(out[0], g * c / math.sqrt(c * c + eps), rtol=0, atol=1e-15)


def test_silu_values():
    assert orc.silu(np.array([0.0]))[0] == 0.0
    assert abs(orc.silu(np.array([1.0]))[0] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    assert abs(orc.silu(np.array([-2.0]))[0] + 2.0 / (1.0 + math.exp(2.0))) < 1e-15


# ---- P8: RoPE ---------------------------------------------------------------------------------
def test_rope_position_zero_identity_and_hand_rotation():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((1, 2, 8))
    assert np.array_equal(orc.rope(x, np.array([0]), 1e6), x)
    # d = 2: a single plane rotated by the angle pos (inv_freq_0 = 1)
    v = np.array([[[1.0, 0.0]]])
    r = orc.rope(v, np.array([1]), 1e6)
    assert np.allclose(r[0, 0], [math.cos(1.0), math.sin(1.0)], atol=1e-15)
    # d = 4, second frequency = theta^(-1/2)
    v = np.array([[[0.0, 1.0, 0.0, 0.0]]])
    r = orc.rope(v, np.array([3]), 100.0)
    assert np.allclose(r[0, 0], [0.0, math.cos(0.3), 0.0, math.sin(0.3)], atol=1e-15)


def test_rope_relative_property_shift_invariance():
    o, _ = make()
    x = np.random.default_rng(1).standard_normal((9, MICRO.hidden))
    a = o.forward_dense(x, orc.causal_mask(9))
    b = o.forward_dense(x, orc.causal_mask(9), positions=np.arange(9) + 1234)
    assert np.abs(a - b).max() < 1e-9
    # ... and positions do matter (a permuted position vector changes the result)
    c = o.forward_dense(x, orc.causal_mask(9), positions=np.arange(9)[::-1])
    assert np.abs(a - c).max() > 1e-4


# ---- P11: independent restatement of attention with a library routine ---------------------------
def test_attend_matches_torch_sdpa():
    rng = np.random.default_rng(2)
    n, T, Hq, Hkv, d = 5, 11, 4, 2, 8
    q, k, v = rng.standard_normal((n, Hq, d)), rng.standard_normal((T, Hkv, d)), rng.standard_normal((T, Hkv, d))
    allowed = rng.random((n, T)) < 0.6
    allowed[:, 0] = True
    got = orc.attend(q, k, v, allowed)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)[None]
    tv = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.from_numpy(allowed)[None, None])
    assert np.abs(ref[0].permute(1, 0, 2).numpy() - got).max() < 1e-12


def test_full_layer_against_torch_restatement():
    """A separately written torch fp64 decoder (library matmul / SDPA / F.silu) on the micro shape."""
    o, w = make(qkv_bias=True)
    s = MICRO
    T = 7
    x = torch.randn(T, s.hidden, dtype=torch.float64, generator=torch.Generator().manual_seed(5))
    h = x.clone()
    pos = torch.arange(T, dtype=torch.float64)
    inv = s.rope_theta ** (-torch.arange(0, s.head_dim, 2, dtype=torch.float64) / s.head_dim)
    ang = pos[:, None] * inv[None]
    cos, sin = torch.cos(ang).repeat(1, 2)[:, None], torch.sin(ang).repeat(1, 2)[:, None]

    def rot(t):
        half = t.shape[-1] // 2
        return t * cos + torch.cat([-t[..., half:], t[..., :half]], -1) * sin

    def norm(t, g):
        return t * torch.rsqrt(t.pow(2).mean(-1, keepdim=True) + s.rms_eps) * g.double()

    for lw in w["layers"]:
        a = norm(h, lw["g_attn"])
        q = (a @ lw["wq"].double().T + lw["bq"].double()).view(T, s.n_q_heads, s.head_dim)
        k = (a @ lw["wk"].double().T + lw["bk"].double()).view(T, s.n_kv_heads, s.head_dim)
        v = (a @ lw["wv"].double().T + lw["bv"].double()).view(T, s.n_kv_heads, s.head_dim)
        q, k = rot(q), rot(k)
        att = torch.nn.functional.scaled_dot_product_attention(
            q.transpose(0, 1)[None], k.transpose(0, 1)[None], v.transpose(0, 1)[None], is_causal=True, enable_gqa=True)
        h = h + att[0].transpose(0, 1).reshape(T, -1) @ lw["wo"].double().T
        m = norm(h, lw["g_mlp"])
        h = h + (torch.nn.functional.silu(m @ lw["w_gate"].double().T) * (m @ lw["w_up"].double().T)) @ lw["w_down"].double().T
    ref = norm(h, w["g_final"]) @ w["embed"].double().T
    hs = o.forward_rows(x.numpy(), orc.CAUSAL, update_cache=True)
    got = o.logits_of(hs)
    assert np.abs(got - ref.numpy()).max() < 1e-10


# ---- P10: zero-layer case checkable by hand --------------------------------------------------------
def test_zero_output_projections_reduce_to_embedding_logits():
    o, w = make()
    for lw in o.w["layers"]:
        lw["wo"] = np.zeros_like(lw["wo"])
        lw["w_down"] = np.zeros_like(lw["w_down"])
    toks = np.array([3, 9, 9, 1])
    o.block_begin(4, toks)
    got = o.block_forward()
    E = w["embed"].double().numpy()
    e = E[toks]
    ref = (e / np.sqrt((e * e).mean(1, keepdims=True) + MICRO.rms_eps)) @ E.T
    assert np.abs(got - ref).max() < 1e-12


# ---- P1: block size 1 is ordinary causal AR decoding ----------------------------------------------
def test_block_size_one_equals_causal_ar():
    o, _ = make()
    emb, toks = prefix(MICRO, 3, 4)
    o.prefill(emb, toks)
    x_prefix = np.concatenate([orc.to_f64(emb), o.embed_tokens(toks)], 0)
    for tok in (5, MICRO.mask_id, 17):
        o.block_begin(1, np.array([tok]))
        row = o.block_forward()[0]
        x = np.concatenate([x_prefix, o.embed_tokens([tok])], 0)
        ref = o.forward_dense(x, orc.causal_mask(len(x)))[-1]
        assert np.abs(row - ref).max() < 1e-10
        o.block_tokens, o.masked = None, None


def test_greedy_ar_via_one_token_commits():
    o, _ = make()
    emb, toks = prefix(MICRO, 2, 3)
    nxt = o.prefill(emb, toks)
    seq_x = np.concatenate([orc.to_f64(emb), o.embed_tokens(toks)], 0)
    for _ in range(4):
        tok = int(np.argmax(nxt[:MICRO.mask_id]))           # the mask token is never generated
        ref = int(np.argmax(o.forward_dense(seq_x, orc.causal_mask(len(seq_x)))[-1][:MICRO.mask_id]))
        assert tok == ref
        o.block_begin(1, np.array([tok]))
        nxt = o.commit_block()
        seq_x = np.concatenate([seq_x, o.embed_tokens([tok])], 0)


# ---- P2: incremental prefill + commit == one dense causal pass -----------------------------------
@pytest.mark.parametrize("chunks", [[9], [4, 5], [1] * 9, [2, 3, 4]])
def test_incremental_prefill_equals_one_shot(chunks):
    o, _ = make()
    emb, toks = prefix(MICRO, 5, 4)
    x = np.concatenate([orc.to_f64(emb), o.embed_tokens(toks)], 0)
    blk = np.array([7, 8, 9])
    x_all = np.concatenate([x, o.embed_tokens(blk)], 0)
    ref = o.forward_dense(x_all, orc.causal_mask(len(x_all)))
    o1, _ = make()
    o1.prefill(emb, toks)
    K_ref = [k.copy() for k in o1.K]
    # chunked: feed rows as embeddings chunk by chunk
    r0 = 0
    last = None
    for c in chunks:
        last = o.prefill(x[r0:r0 + c], None)
        r0 += c
    assert np.abs(last - ref[len(x) - 1]).max() < 1e-10
    for a, b in zip(o.K, K_ref):
        assert np.abs(a - b).max() < 1e-12
    o.block_begin(3, blk)
    nxt = o.commit_block()
    assert o.cache_len == len(x_all)
    assert np.abs(nxt - ref[-1]).max() < 1e-10


# ---- P3: the cached path equals a brute-force dense mask (Alg. 2 step-1 mask / lower triangle) ----
@pytest.mark.parametrize("L", [0, 1, 3])
@pytest.mark.parametrize("B", [1, 2, 3, 5])
@pytest.mark.parametrize("heads", [(4, 4), (4, 2), (4, 1)])
def test_cached_path_equals_bruteforce_mask(L, B, heads):
    shape = MICRO.with_(n_q_heads=heads[0], n_kv_heads=heads[1], n_layers=1)
    o, _ = make(shape, seed=11)
    toks = I.random_tokens(shape, L + B, 21).numpy()
    if L:
        o.prefill(None, toks[:L])
    blk = toks[L:].copy()
    blk[B // 2:] = shape.mask_id
    o.block_begin(B, blk)
    got = o.block_forward()
    x = o.embed_tokens(np.concatenate([toks[:L], blk]))
    ref = o.forward_dense(x, orc.draft_mask(L, B))[L:]
    assert np.abs(got - ref).max() < 1e-10
    # commit mode: lower-triangular everywhere
    h = o.forward_rows(o.embed_tokens(blk), orc.CAUSAL, update_cache=False)
    ref_c = o.forward_dense(x, orc.causal_mask(L + B))[L:]
    assert np.abs(o.logits_of(h) - ref_c).max() < 1e-10


def test_draft_mask_definition():
    m = orc.draft_mask(2, 2)
    assert m.tolist() == [[True, False, False, False], [True, True, False, False],
                          [True, True, True, True], [True, True, True, True]]


# ---- P4: dependency probes --------------------------------------------------------------------------
def test_dependency_structure_and_cache_untouched_by_steps():
    o, _ = make()
    emb, toks = prefix(MICRO, 3, 3)
    o.prefill(emb, toks)
    K0 = [k.copy() for k in o.K]
    V0 = [v.copy() for v in o.V]
    blk = np.array([1, 2, 3, 4, 5])
    o.block_begin(5, blk)
    base = o.block_forward()
    blk2 = blk.copy()
    blk2[3] = 40
    o.block_begin(5, blk2)
    pert = o.block_forward()
    assert all(np.abs(base[i] - pert[i]).max() > 1e-9 for i in range(5))        # bidirectional: all rows move
    hc = o.logits_of(o.forward_rows(o.embed_tokens(blk), orc.CAUSAL, False))
    hp = o.logits_of(o.forward_rows(o.embed_tokens(blk2), orc.CAUSAL, False))
    assert np.array_equal(hc[:3], hp[:3]) and np.abs(hc[3:] - hp[3:]).max() > 1e-9  # causal: rows < 3 fixed
    o.block_begin(5)
    while o.masked.any():
        o.block_step(orc.THRESHOLD, 0.9)
    assert o.cache_len == 6
    assert all(np.array_equal(a, b) for a, b in zip(o.K, K0)) and all(np.array_equal(a, b) for a, b in zip(o.V, V0))


# ---- P5: selection closed forms ----------------------------------------------------------------------
def test_selection_threshold_rules():
    conf = np.array([0.95, 0.2, 0.91, 0.9, 0.5])
    masked = np.array([True, True, True, True, False])
    assert orc.select_unmask(conf, masked, orc.THRESHOLD, 0.9).tolist() == [True, False, True, False, False]
    # nothing above tau -> exactly the most confident masked position (position 4 is not masked)
    c2 = np.array([0.1, 0.3, 0.2, 0.3, 0.99])
    assert orc.select_unmask(c2, masked, orc.THRESHOLD, 0.9).tolist() == [False, True, False, False, False]
    # tau = 1.0: strict inequality, a saturated confidence still reveals one token only
    c3 = np.array([1.0, 1.0, 0.5, 0.2, 0.1])
    assert orc.select_unmask(c3, masked, orc.THRESHOLD, 1.0).sum() == 1
    # tau < 0: everything masked is revealed in one step
    assert orc.select_unmask(conf, masked, orc.THRESHOLD, -1.0).tolist() == masked.tolist()
    assert orc.select_unmask(conf, np.zeros(5, bool), orc.THRESHOLD, 0.5).sum() == 0


def test_selection_topk_rules():
    conf = np.array([0.3, 0.9, 0.3, 0.8, 0.1, 0.7])
    masked = np.array([True, True, True, True, True, False])
    assert orc.select_unmask(conf, masked, orc.TOPK, k=2).tolist() == [False, True, False, True, False, False]
    assert orc.select_unmask(conf, masked, orc.TOPK, k=3).tolist() == [True, True, False, True, False, False]  # tie -> lower index
    assert orc.select_unmask(conf, masked, orc.TOPK, k=9).tolist() == masked.tolist()


@pytest.mark.parametrize("rule,tau,k,B,expect", [
    (orc.THRESHOLD, 1.0, 0, 6, [1] * 6),          # Sec. 4.5: tau = 1.0 -> one token per step
    (orc.THRESHOLD, -1.0, 0, 6, [6]),             # draft: every mask filled in one pass
    (orc.TOPK, 0.0, 8, 32, [8, 8, 8, 8]),
    (orc.TOPK, 0.0, 4, 10, [4, 4, 2]),
])
def test_decode_loop_step_counts_and_termination(rule, tau, k, B, expect):
    o, _ = make()
    emb, toks = prefix(MICRO, 2, 2)
    o.prefill(emb, toks)
    steps, _ = o.decode_block(B, rule, tau, k)
    assert [s["n_unmasked"] for s in steps] == expect
    assert steps[-1]["n_remaining"] == 0 and MICRO.mask_id not in steps[-1]["block_tokens"]
    assert o.cache_len == 4 + B


def test_threshold_loop_invariants_peaked_model():
    o, _ = make(final_gain=40.0)
    o.prefill(None, np.array([1, 2, 3]))
    steps, _ = o.decode_block(12, orc.THRESHOLD, 0.9)
    assert 1 <= len(steps) <= 12 and all(s["n_unmasked"] >= 1 for s in steps)
    assert sum(s["n_unmasked"] for s in steps) == 12
    for s in steps:   # only masked positions are revealed, with their own prediction
        assert not (s["unmask"] & ~s["masked_before"]).any()
        assert np.array_equal(s["block_tokens"][s["unmask"]], s["pred"][s["unmask"]])
        hit = s["masked_before"] & (s["conf"] > 0.9)
        assert np.array_equal(s["unmask"], hit) if hit.any() else s["unmask"].sum() == 1
    assert any(s["n_unmasked"] > 1 for s in steps) or len(steps) == 12


# ---- P6: softmax / confidence identities ------------------------------------------------------------
def test_confidence_identities():
    rng = np.random.default_rng(4)
    V, mid = 50, 49
    l = rng.standard_normal((6, V)) * 3
    l[2, mid] = 100.0                                   # the mask token may never win
    pred, conf, margin = orc.confidence(l, mid)
    lm = l.copy()
    lm[:, mid] = -np.inf
    p = np.exp(lm - lm.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    assert np.allclose(p.sum(1), 1.0) and np.allclose(conf, p.max(1), atol=1e-15)
    assert (pred != mid).all() and np.array_equal(pred, p.argmax(1))
    assert (conf >= 1.0 / (V - 1) - 1e-15).all() and (conf <= 1.0).all()
    srt = np.sort(p, axis=1)
    assert np.allclose(margin, srt[:, -1] - srt[:, -2], atol=1e-15)
    # uniform logits: conf = 1/(V-1), lowest id wins the tie
    pred, conf, _ = orc.confidence(np.zeros((1, V)), mid)
    assert pred[0] == 0 and abs(conf[0] - 1.0 / (V - 1)) < 1e-15


# ---- P7: GQA == MHA with repeated K/V weights --------------------------------------------------------
def test_gqa_equals_mha_with_repeated_kv_weights():
    o, w = make(qkv_bias=True)
    s2 = MICRO.with_(n_kv_heads=MICRO.n_q_heads)
    grp = MICRO.n_q_heads // MICRO.n_kv_heads
    wn = I.weights_to_numpy(w)
    for lw in wn["layers"]:
        for name in ("wk", "wv"):
            lw[name] = np.repeat(lw[name].reshape(MICRO.n_kv_heads, MICRO.head_dim, -1), grp, axis=0).reshape(-1, MICRO.hidden)
        for name in ("bk", "bv"):
            lw[name] = np.repeat(lw[name].reshape(MICRO.n_kv_heads, MICRO.head_dim), grp, axis=0).reshape(-1)
    o2 = orc.Oracle(s2, wn)
    toks = np.array([4, 5, 6, 7])
    for m in (o, o2):
        m.prefill(None, toks)
        m.block_begin(3)
    assert np.abs(o.block_forward() - o2.block_forward()).max() < 1e-10


# ---- P12: the oracle's own rounding is far below the GPU tolerances -----------------------------------
def test_fp32_oracle_close_to_fp64_oracle():
    w = I.make_weights(I.TINY, 0)
    wn = I.weights_to_numpy(w)
    emb, toks = I.make_prefix(I.TINY, 48, 16, 10)
    outs = []
    for ft in (np.float64, np.float32):
        o = orc.Oracle(I.TINY, wn, ftype=ft)
        o.prefill(I.as_numpy_storage(emb), toks.numpy())
        o.block_begin(8)
        outs.append(np.asarray(o.block_forward(), dtype=np.float64))
    assert np.abs(outs[0] - outs[1]).max() < 1e-5


# ---- FP8 storage with per-output-channel scales, and the untied LM head -----------------------------
def _hand_e4m3():
    """A 2 x 3 e4m3 matrix written out code by code (sign | 4 exponent bits, bias 7 | 3 mantissa bits) with one scale per
    ROW (= output channel), and its value worked by hand."""
    codes = np.array([[0x38, 0x40, 0xB8],        #  1.0   2.0   -1.0
                      [0x3C, 0x30, 0x7E]],       #  1.5   0.5   448 (largest finite)
                     dtype=np.uint8)
    scales = np.array([0.5, 3.0], dtype=np.float32)
    value = [[0.5, 1.0, -0.5], [4.5, 1.5, 1344.0]]
    return codes, scales, value


def test_fp8_weight_with_row_scales_by_hand():
    codes, scales, value = _hand_e4m3()
    o = orc.Oracle(MICRO, {"layers": [{"wq": codes, "s_q": scales}]})
    w = o._lin(0, "wq")
    assert w.shape == (2, 3)
    for r in range(2):
        for c in range(3):
            assert w[r, c] == value[r][c], (r, c, w[r, c])
    # orientation in a projection: [out, in], so a one-hot input picks a COLUMN of the matrix
    assert np.array_equal(np.array([0.0, 1.0, 0.0]) @ w.T, [1.0, 1.5])
    # a matrix without scales is taken as stored
    assert np.array_equal(orc.Oracle(MICRO, {"layers": [{"wq": codes}]})._lin(0, "wq"), [[1.0, 2.0, -1.0], [1.5, 0.5, 448.0]])


FP8_MICRO = MICRO.with_(dtype=I.FP8, tie_embeddings=False)


def _untied_logits_by_hand(o, w, h):
    """RMSNorm(h; g_final) . (e4m3(lm_head) * s_lm_head[row])^T with plain Python loops and torch's own e4m3 cast."""
    shape = o.s
    table = w["lm_head"].view(torch.float8_e4m3fn).to(torch.float64).numpy()
    s_head = w["s_lm_head"].double().numpy()
    g = w["g_final"].double().numpy()
    out = np.zeros((h.shape[0], shape.vocab))
    for r in range(h.shape[0]):
        ms = sum(float(v) ** 2 for v in h[r]) / shape.hidden
        a = [float(h[r, c]) / math.sqrt(ms + shape.rms_eps) * g[c] for c in range(shape.hidden)]
        for v in range(shape.vocab):
            out[r, v] = sum(a[c] * table[v, c] * s_head[v] for c in range(shape.hidden))
    return out


def test_untied_fp8_lm_head_row_by_row():
    o, w = make(FP8_MICRO, seed=5, final_gain=1.7)
    assert w["lm_head"] is not None and w["lm_head"].dtype == torch.uint8 and w["s_lm_head"].shape == (FP8_MICRO.vocab,)
    # the scales must differ from row to row for the test to see a wrong axis
    assert len(set(np.round(w["s_lm_head"].numpy(), 9).tolist())) > FP8_MICRO.vocab // 2
    h = np.random.default_rng(1).standard_normal((3, FP8_MICRO.hidden))
    got = o.logits_of(h)
    want = _untied_logits_by_hand(o, w, h)
    assert np.abs(got - want).max() < 1e-12
    # and the embedding table plays no part in an untied head
    o.w["embed"] = np.zeros_like(o.w["embed"])
    assert np.array_equal(o.logits_of(h), got)


def test_fp8_micro_model_layer_matmuls_use_row_scales():
    """A whole forward of the FP8 micro model against the torch restatement fed with explicitly de-quantised weights
    (value = e4m3 code * scale of its output row), so every projection's scale handling is covered."""
    o, w = make(FP8_MICRO, seed=6)
    deq = {"embed": w["embed"].double(), "g_final": w["g_final"].double(),
           "lm_head": w["lm_head"].view(torch.float8_e4m3fn).double() * w["s_lm_head"].double()[:, None], "layers": []}
    for lw in w["layers"]:
        d = {}
        for name, sname in (("wq", "s_q"), ("wk", "s_k"), ("wv", "s_v"), ("wo", "s_o"), ("w_gate", "s_gate"), ("w_up", "s_up"),
                            ("w_down", "s_down")):
            d[name] = lw[name].view(torch.float8_e4m3fn).double() * lw[sname].double()[:, None]
        deq["layers"].append(d)
    s = FP8_MICRO
    toks = torch.tensor([3, 9, 27, 5, 11])
    h = deq["embed"][toks]
    T = len(toks)
    pos = torch.arange(T, dtype=torch.float64)
    half = s.head_dim // 2
    inv = s.rope_theta ** (-torch.arange(half, dtype=torch.float64) * 2 / s.head_dim)
    cos, sin = torch.cos(pos[:, None] * inv), torch.sin(pos[:, None] * inv)

    def rot(x):
        x1, x2 = x[..., :half], x[..., half:]
        return torch.cat([x1 * cos[:, None] - x2 * sin[:, None], x2 * cos[:, None] + x1 * sin[:, None]], -1)

    def norm(x):
        return x / torch.sqrt((x * x).mean(-1, keepdim=True) + s.rms_eps)
    for d in deq["layers"]:
        a = norm(h)
        q = rot((a @ d["wq"].T).view(T, s.n_q_heads, s.head_dim))
        k = rot((a @ d["wk"].T).view(T, s.n_kv_heads, s.head_dim))
        v = (a @ d["wv"].T).view(T, s.n_kv_heads, s.head_dim)
        rep = s.n_q_heads // s.n_kv_heads
        att = torch.nn.functional.scaled_dot_product_attention(q.transpose(0, 1), k.repeat_interleave(rep, 1).transpose(0, 1),
                                                               v.repeat_interleave(rep, 1).transpose(0, 1), is_causal=True)
        h = h + att.transpose(0, 1).reshape(T, -1) @ d["wo"].T
        m = norm(h)
        h = h + (torch.nn.functional.silu(m @ d["w_gate"].T) * (m @ d["w_up"].T)) @ d["w_down"].T
    want = (norm(h) * deq["g_final"]) @ deq["lm_head"].T
    got = o.prefill(None, toks.numpy())
    assert np.abs(got - want[-1].numpy()).max() < 1e-10


# ---- planted mistakes must be caught: each plants one plausible error in the oracle and requires a pin above to FAIL ----
def _must_fail(pin, *args):
    try:
        pin(*args)
    except AssertionError:
        return
    raise AssertionError(f"{pin.__name__} did not notice the planted error")


def test_planted_rope_sign_error_fails_the_hand_rotation_pin(monkeypatch):
    good = orc.rope
    monkeypatch.setattr(orc, "rope", lambda x, pos, theta: good(x, -np.asarray(pos), theta))
    _must_fail(test_rope_position_zero_identity_and_hand_rotation)


def test_planted_scale_on_the_wrong_axis_fails_the_fp8_pins(monkeypatch):
    def bad_lin(self, layer, name):
        lw = self.w["layers"][layer]
        w = orc.to_f64(lw[name])
        sc = lw.get({"wq": "s_q", "wk": "s_k", "wv": "s_v", "wo": "s_o", "w_gate": "s_gate", "w_up": "s_up", "w_down": "s_down"}[name])
        if sc is not None:
            n = min(w.shape)
            w = w.copy()
            w[:n, :n] = w[:n, :n] * orc.to_f64(sc)[None, :n]          # per INPUT column instead of per output row
        return w
    monkeypatch.setattr(orc.Oracle, "_lin", bad_lin)
    _must_fail(test_fp8_weight_with_row_scales_by_hand)
    _must_fail(test_fp8_micro_model_layer_matmuls_use_row_scales)


def test_planted_ignored_lm_head_fails_the_untied_pin(monkeypatch):
    good = orc.Oracle.logits_of

    def bad(self, h, chunk=16384):
        saved = self.w.get("lm_head")
        self.w["lm_head"] = None                                     # falls back to the embedding table
        try:
            return good(self, h, chunk)
        finally:
            self.w["lm_head"] = saved
    monkeypatch.setattr(orc.Oracle, "logits_of", bad)
    _must_fail(test_untied_fp8_lm_head_row_by_row)


def test_planted_ignored_head_scale_fails_the_untied_pin(monkeypatch):
    good = orc.Oracle.logits_of

    def bad(self, h, chunk=16384):
        saved = self.w.get("s_lm_head")
        self.w["s_lm_head"] = None
        try:
            return good(self, h, chunk)
        finally:
            self.w["s_lm_head"] = saved
    monkeypatch.setattr(orc.Oracle, "logits_of", bad)
    _must_fail(test_untied_fp8_lm_head_row_by_row)
