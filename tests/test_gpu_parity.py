"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Tolerances: fp32 1e-4 (logits and confidence); bf16 3e-2 / 5e-3; fp8 weights 8e-2 / 1e-2.
Token ids must agree where the oracle's top-2 probability margin exceeds 1e-3; unmask sets and step
counts where every selection decision is clear of the confidence tolerance."""
import numpy as np
import pytest
import torch

from oracle import fdvlm_oracle as orc
from paper_2604_06832_b200 import inputs as I

from helpers import TOL, make_pair, replay_decode, upload_prefix

pytestmark = pytest.mark.gpu

SMALL_BF16 = I.ModelShape(n_layers=3, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, intermediate=1376,
                          vocab=4096, mask_id=4095, tie_embeddings=True, dtype=I.BF16)
SMALL_FP8 = SMALL_BF16.with_(dtype=I.FP8, tie_embeddings=False, n_q_heads=4, n_kv_heads=4, head_dim=64, hidden=384,
                             intermediate=1120, vocab=3000, mask_id=2999)


def B():
    from paper_2604_06832_b200 import binding
    return binding


# ---- single operators -------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [I.F32, I.BF16, I.FP8])
@pytest.mark.parametrize("m,n,k", [(1, 64, 64), (8, 200, 688), (32, 2560, 2048), (33, 1000, 1376), (64, 4096, 512),
                                   (5, 72, 2048), (32, 2048, 11008)])
def test_op_linear_matches_oracle_matmul(dtype, m, n, k):
    g = torch.Generator().manual_seed(m * 1000 + n + k)
    x = torch.randn(m, k, generator=g)
    w = torch.randn(n, k, generator=g) * 0.05
    bias = torch.randn(n, generator=g) * 0.1
    if dtype == I.F32:
        xs, ws, sc = x, w, None
        xv, wv = x.double().numpy(), w.double().numpy()
    else:
        xs = x.to(torch.bfloat16)
        xv = orc.to_f64(I.as_numpy_storage(xs))
        if dtype == I.BF16:
            ws, sc = w.to(torch.bfloat16), None
            wv = orc.to_f64(I.as_numpy_storage(ws))
        else:
            ws, sc = I.quantize_e4m3_rows(w)
            wv = orc.to_f64(ws.numpy()) * sc.double().numpy()[:, None]
    ref = xv @ wv.T + bias.double().numpy()
    code = {I.F32: B().DT_F32, I.BF16: B().DT_BF16, I.FP8: B().DT_FP8}[dtype]
    y = B().op_linear(xs.cuda(), ws.cuda(), None if sc is None else sc.cuda(), bias.cuda(), dtype=code)
    torch.cuda.synchronize()
    err = np.abs(y.double().cpu().numpy() - ref).max()
    scale = np.abs(ref).max()
    assert err <= (2e-5 if dtype == I.F32 else 2e-4) * max(scale, 1.0), (err, scale)   # fp32 accumulation of exact products


@pytest.mark.parametrize("dtype", [I.F32, I.BF16, "f16"])
@pytest.mark.parametrize("n,L,hq,hkv,d,causal", [(1, 0, 4, 2, 64, 0), (8, 64, 4, 2, 64, 0), (8, 64, 4, 2, 64, 1),
                                                 (32, 1000, 16, 2, 128, 0), (32, 1000, 16, 2, 128, 1),
                                                 (5, 3, 4, 4, 128, 1), (64, 517, 8, 1, 128, 0), (17, 2100, 28, 4, 128, 0)])
def test_op_attention_matches_oracle(dtype, n, L, hq, hkv, d, causal):
    g = torch.Generator().manual_seed(n + L + hq)
    max_seq = L + n + 7
    td = {I.F32: torch.float32, I.BF16: torch.bfloat16, "f16": torch.float16}[dtype]
    q = torch.randn(n, hq, d, generator=g).to(td)
    kc = torch.randn(hkv, max_seq, d, generator=g).to(td)
    vc = torch.randn(hkv, max_seq, d, generator=g).to(td)
    T = L + n
    allowed = np.ones((n, T), dtype=bool)
    if causal:
        allowed[:, L:] = np.tril(np.ones((n, n), dtype=bool))
    f = lambda t: t.double().numpy()          # the exact value of every storage type
    ref = orc.attend(f(q), f(kc)[:, :T].transpose(1, 0, 2), f(vc)[:, :T].transpose(1, 0, 2), allowed).reshape(n, hq * d)
    out = B().op_attention(q.cuda(), kc.cuda(), vc.cuda(), L, bool(causal), dtype=B().DT_F32 if dtype == I.F32 else B().DT_BF16)
    torch.cuda.synchronize()
    err = np.abs(out.double().cpu().numpy() - ref).max()
    # the probabilities and the result are rounded to the element type: 2^-9 relative for bf16, 2^-12 for f16
    assert err <= {I.F32: 2e-5, I.BF16: 2e-2, "f16": 3e-3}[dtype], err


# ---- configuration 1: tiny fp32, the full decode of one block of 8 at threshold 0.9 ------------------
def test_cfg1_tiny_fp32_full_decode():
    wl = I.WORKLOADS["cfg1_tiny_f32"]
    oracle, handle, _ = make_pair(wl.shape, wl.weight_seed, max_seq=128)
    emb, toks = I.make_prefix(wl.shape, wl.n_embeds, wl.n_tokens, wl.prefix_seed)
    ref_last = oracle.prefill(I.as_numpy_storage(emb), toks.numpy())
    last = torch.empty(wl.shape.vocab, dtype=torch.float32, device="cuda")
    e, t = upload_prefix(emb, toks)
    handle.prefill(e, t, last)
    assert handle.cache_len() == 64
    assert np.abs(last.double().cpu().numpy() - ref_last).max() <= 1e-4
    for layer in range(wl.shape.n_layers):
        for which, ref in ((0, oracle.K[layer]), (1, oracle.V[layer])):
            got = handle.cache_read(layer, which, 0, 64).double().cpu().numpy()
            assert np.abs(got - ref).max() <= 1e-4
    stats = replay_decode(oracle, handle, wl.shape, 8, orc.THRESHOLD, wl.threshold)
    assert stats["steps"] == 8 and handle.cache_len() == 72
    # free-running (no replay): the same 8-step structure, no masks left
    handle.block_begin(8)
    tokens = torch.empty(8, dtype=torch.int32, device="cuda")
    n_steps = 0
    while True:
        info = handle.block_step(B().RULE_THRESHOLD, 0.9, block_tokens=tokens)
        n_steps += 1
        assert info.n_unmasked >= 1 and info.step_index == n_steps
        if info.n_remaining == 0:
            break
    assert n_steps <= 8 and (tokens.cpu().numpy() != wl.shape.mask_id).all()
    handle.commit_block()
    assert handle.cache_len() == 80
    handle.close()


@pytest.mark.parametrize("chunks", [[64], [10, 54], [1, 1, 62]])
def test_cfg1_prefill_chunking_is_equivalent(chunks):
    wl = I.WORKLOADS["cfg1_tiny_f32"]
    oracle, handle, _ = make_pair(wl.shape, wl.weight_seed, max_seq=128, max_block=16)
    emb, toks = I.make_prefix(wl.shape, wl.n_embeds, wl.n_tokens, wl.prefix_seed)
    ref_last = oracle.prefill(I.as_numpy_storage(emb), toks.numpy())
    rows = torch.cat([emb, I.make_weights(wl.shape, wl.weight_seed)["embed"][toks.long()]], 0).cuda()
    last = torch.empty(wl.shape.vocab, dtype=torch.float32, device="cuda")
    r0 = 0
    for c in chunks:
        handle.prefill(rows[r0:r0 + c].contiguous(), None, last)
        r0 += c
    assert np.abs(last.double().cpu().numpy() - ref_last).max() <= 1e-4
    handle.close()


# ---- peaked tiny model: confidences spread over (0,1), so the discrete decisions are really exercised --
@pytest.mark.parametrize("rule,tau,k,B_", [(orc.THRESHOLD, 0.9, 0, 8), (orc.THRESHOLD, 0.5, 0, 16), (orc.TOPK, 0.0, 3, 8),
                                          (orc.THRESHOLD, 1.0, 0, 5), (orc.THRESHOLD, -1.0, 0, 7)])
def test_tiny_fp32_peaked_discrete_parity(rule, tau, k, B_):
    wl = I.WORKLOADS["cfg1_tiny_f32"]
    oracle, handle, _ = make_pair(wl.shape, wl.weight_seed, max_seq=160, final_gain=24.0)
    emb, toks = I.make_prefix(wl.shape, wl.n_embeds, wl.n_tokens, wl.prefix_seed)
    oracle.prefill(I.as_numpy_storage(emb), toks.numpy(), want_logits=False)
    handle.prefill(*upload_prefix(emb, toks))
    stats = replay_decode(oracle, handle, wl.shape, B_, rule, tau, k, n_blocks=2, tol=dict(logits=2e-3, conf=1e-4, gap=4e-3))
    assert stats.get("rows_sure", 0) > 0 and stats.get("steps_clear", 0) > 0
    handle.close()


# ---- bf16 / fp8 small shapes (ragged sizes, biases) ------------------------------------------------------
@pytest.mark.parametrize("shape,B_,L_e,L_t,rule,k", [
    (SMALL_BF16, 32, 70, 31, orc.TOPK, 8),
    (SMALL_BF16, 5, 0, 9, orc.THRESHOLD, 0),
    (SMALL_BF16.with_(head_dim=64, n_q_heads=4, n_kv_heads=4), 16, 40, 0, orc.TOPK, 5),
    (SMALL_FP8, 32, 33, 40, orc.TOPK, 8),
    (SMALL_FP8.with_(tie_embeddings=True), 7, 20, 20, orc.THRESHOLD, 0),
])
@pytest.mark.parametrize("kv", ["f16", "bf16"])
def test_small_bf16_fp8_parity(shape, B_, L_e, L_t, rule, k, kv):
    oracle, handle, _ = make_pair(shape, 7, max_seq=256, qkv_bias=True, kv_dtype=B().KV_F16 if kv == "f16" else B().KV_BF16)
    emb, toks = I.make_prefix(shape, L_e, L_t, 3)
    ref_last = oracle.prefill(I.as_numpy_storage(emb) if L_e else None, toks.numpy() if L_t else None)
    last = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
    handle.prefill(*upload_prefix(emb, toks), last)
    tol = TOL[shape.dtype]
    assert np.abs(last.double().cpu().numpy() - ref_last).max() <= tol["logits"]
    stats = replay_decode(oracle, handle, shape, B_, rule, 0.9, k, n_blocks=2)
    assert stats["steps"] >= 2
    handle.close()


@pytest.mark.parametrize("shape,B_", [(SMALL_BF16, 32), (SMALL_BF16, 5), (SMALL_FP8, 16)])
def test_parity_through_captured_graphs_on_a_user_stream(shape, B_):
    """On a caller-given stream the forward is replayed from CUDA graphs captured once per (rows, mode): several blocks
    at growing cache lengths must keep matching the oracle (the cache length travels through device memory)."""
    stream = torch.cuda.Stream()
    oracle, handle, _ = make_pair(shape, 21, max_seq=400, stream=stream, qkv_bias=True)
    emb, toks = I.make_prefix(shape, 37, 30, 6)
    ref_last = oracle.prefill(I.as_numpy_storage(emb), toks.numpy())
    last = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
    with torch.cuda.stream(stream):
        handle.prefill(*upload_prefix(emb, toks), last)
        stream.synchronize()
        assert np.abs(last.double().cpu().numpy() - ref_last).max() <= TOL[shape.dtype]["logits"]
        stats = replay_decode(oracle, handle, shape, B_, orc.TOPK, 0.9, 4, n_blocks=3)
    assert stats["steps"] >= 3 and handle.cache_len() == 67 + 3 * B_
    handle.close()


def test_small_bf16_peaked_discrete_parity():
    oracle, handle, _ = make_pair(SMALL_BF16, 9, max_seq=256, final_gain=16.0)
    emb, toks = I.make_prefix(SMALL_BF16, 20, 20, 4)
    oracle.prefill(I.as_numpy_storage(emb), toks.numpy(), want_logits=False)
    handle.prefill(*upload_prefix(emb, toks))
    stats = replay_decode(oracle, handle, SMALL_BF16, 32, orc.THRESHOLD, 0.9, n_blocks=1, tol=dict(gap=2 * TOL[I.BF16]["logits"], **TOL[I.BF16]))     # the stated bf16 bounds, although the final gain is 16
    print("peaked small bf16:", stats)
    assert stats.get("rows_sure", 0) > 100 and stats.get("steps_clear", 0) > 0
    handle.close()


# ---- invariants on the GPU side ---------------------------------------------------------------------------
def test_steps_do_not_touch_committed_cache_and_are_deterministic():
    oracle, handle, _ = make_pair(SMALL_BF16, 11, max_seq=128)
    emb, toks = I.make_prefix(SMALL_BF16, 30, 10, 5)
    handle.prefill(*upload_prefix(emb, toks))
    before = [handle.cache_read(l, w, 0, 40).clone() for l in range(3) for w in (0, 1)]
    lg = [torch.empty(16, SMALL_BF16.vocab, dtype=torch.float32, device="cuda") for _ in range(2)]
    for i in range(2):
        handle.block_begin(16)
        handle.block_step(B().RULE_TOPK, 0.0, 4, logits=lg[i])
        handle.block_step(B().RULE_TOPK, 0.0, 4)
        # abandon the block: reset the state machine by re-prefilling from scratch on the second round
        after = [handle.cache_read(l, w, 0, 40) for l in range(3) for w in (0, 1)]
        assert all(torch.equal(a, b) for a, b in zip(before, after))
        handle.reset()
        handle.prefill(*upload_prefix(emb, toks))
    assert torch.equal(lg[0], lg[1])
    handle.close()


def test_state_machine_errors_on_device():
    b = B()
    _, handle, _ = make_pair(I.TINY, 0, max_seq=40, max_block=8)
    with pytest.raises(b.FdvlmError) as e:
        handle.block_step(b.RULE_THRESHOLD)
    assert e.value.code == b.ERR_STATE
    with pytest.raises(b.FdvlmError) as e:
        handle.commit_block()
    assert e.value.code == b.ERR_STATE
    with pytest.raises(b.FdvlmError) as e:
        handle.block_begin(9)
    assert e.value.code == b.ERR_CAPACITY
    toks = I.random_tokens(I.TINY, 36, 1).cuda()
    handle.prefill(None, toks)
    with pytest.raises(b.FdvlmError) as e:
        handle.block_begin(8)                     # 36 + 8 > 40
    assert e.value.code == b.ERR_CAPACITY
    handle.block_begin(4)
    with pytest.raises(b.FdvlmError) as e:
        handle.block_begin(4)
    assert e.value.code == b.ERR_STATE
    with pytest.raises(b.FdvlmError) as e:
        handle.commit_block()                     # masks left
    assert e.value.code == b.ERR_STATE
    with pytest.raises(b.FdvlmError) as e:
        handle.prefill(None, toks[:1])
    assert e.value.code == b.ERR_STATE
    info = handle.block_step(b.RULE_THRESHOLD, -1.0)
    assert info.n_remaining == 0 and info.n_unmasked == 4
    with pytest.raises(b.FdvlmError) as e:
        handle.block_step(b.RULE_THRESHOLD)
    assert e.value.code == b.ERR_STATE
    handle.commit_block()
    assert handle.cache_len() == 40
    handle.close()


def test_host_buffer_variants_match_device_variants():
    b = B()
    _, handle, _ = make_pair(I.TINY, 0, max_seq=64, max_block=8)
    toks = I.random_tokens(I.TINY, 10, 2)
    handle.prefill(None, toks.cuda())
    init = torch.full((8,), I.TINY.mask_id, dtype=torch.int32)
    init[0] = 17
    conf_d = torch.empty(8, dtype=torch.float32, device="cuda")
    pred_d = torch.empty(8, dtype=torch.int32, device="cuda")
    handle.block_begin(8, init.cuda())
    i1 = handle.block_step(b.RULE_TOPK, 0.0, 3, conf=conf_d, pred=pred_d)
    handle.reset()
    handle.prefill(None, toks.cuda())
    conf_h, pred_h = torch.empty(8, dtype=torch.float32), torch.empty(8, dtype=torch.int32)
    um_h, tok_h = torch.empty(8, dtype=torch.uint8), torch.empty(8, dtype=torch.int32)
    handle.block_begin_host(8, init)
    i2 = handle.block_step_host(b.RULE_TOPK, 0.0, 3, conf=conf_h, pred=pred_h, unmask=um_h, block_tokens=tok_h)
    assert (i1.n_unmasked, i1.n_remaining) == (i2.n_unmasked, i2.n_remaining) == (3, 4)
    assert torch.equal(conf_d.cpu(), conf_h) and torch.equal(pred_d.cpu(), pred_h)
    assert tok_h[0] == 17 and um_h[0] == 0 and um_h.sum() == 3
    handle.close()


def test_fp8_weight_codes_are_widened_exactly():
    # one-hot activation rows pick single weights: the output must be the decoded e4m3 value times the row scale,
    # bit for bit, for every finite code (normals, subnormals, both zeros)
    b = B()
    codes = np.array([c for c in range(256) if c not in (0x7F, 0xFF)], dtype=np.uint8)
    n, k, m = 128, 256, 32
    rng = np.random.default_rng(0)
    w = rng.choice(codes, size=(n, k)).astype(np.uint8)
    w[:, :254] = codes[None, :]                      # every code in every row
    cols = rng.choice(k, size=m, replace=False)
    cols[:8] = [0, 1, 7, 8, 0x78, 0x80 - 1, 200, 253]
    x = np.zeros((m, k), dtype=np.float32)
    x[np.arange(m), cols] = 1.0
    scale = (2.0 ** rng.integers(-3, 3, size=n)).astype(np.float32)      # powers of two keep the product exact
    y = b.op_linear(torch.from_numpy(x).to(torch.bfloat16).cuda(), torch.from_numpy(w).cuda(), torch.from_numpy(scale).cuda(),
                    None, dtype=b.DT_FP8).cpu().numpy()
    want = (orc.decode_e4m3(w)[:, cols] * scale[:, None].astype(np.float64)).T
    assert np.array_equal(y.astype(np.float64), want)


# ---- edge sizes: single-row and maximum blocks (every activation-tile width of the GEMM: 16, 32, 48, 64 rows), an
# ---- empty cache, and a decode that ends exactly at max_seq ------------------------------------------------------
@pytest.mark.parametrize("shape,B_,L_t", [(SMALL_BF16, 1, 9), (SMALL_BF16, 40, 17), (SMALL_BF16, 64, 30), (SMALL_FP8, 64, 12),
                                          (SMALL_FP8, 48, 5), (SMALL_BF16, 16, 0), (SMALL_FP8, 3, 0)])
def test_edge_block_sizes_and_empty_cache(shape, B_, L_t):
    n_blocks = 2
    oracle, handle, _ = make_pair(shape, 13, max_seq=L_t + n_blocks * B_, max_block=B_)      # the last commit fills the cache
    if L_t:
        toks = I.random_tokens(shape, L_t, 6)
        oracle.prefill(None, toks.numpy(), want_logits=False)
        handle.prefill(None, toks.cuda())
    stats = replay_decode(oracle, handle, shape, B_, orc.TOPK, 0.9, 7, n_blocks=n_blocks)
    assert stats["steps"] == n_blocks * -(-B_ // 7) and handle.cache_len() == L_t + n_blocks * B_
    with pytest.raises(B().FdvlmError) as e:
        handle.block_begin(1)                            # the cache is full
    assert e.value.code == B().ERR_CAPACITY
    handle.close()
