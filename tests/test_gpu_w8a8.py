"""GPU parity of the W8A8 path (Sec. 3.4 "System integration", Sec. 4.5): fp8 weights and per-token fp8 inputs of the four
layer projections.

Two kinds of check, because a quantiser is a step function.  (1) Where both sides quantise the SAME numbers -- the
stand-alone projection, whose input rows are stored as f16 first -- every e4m3 code is decided identically (float32
quotient, round to nearest even), so the products are exact and the result must agree to fp32 summation error.
(2) Through a whole model the two sides reach each quantiser with inputs that differ in the last bits (fp32 sums and
f16 storage against fp64), a few codes land on the other side of a rounding boundary, each such code moves by a whole
e4m3 spacing (2^-3 .. 2^-4 relative), and the following quantisers amplify the difference again: after a few layers
two correct implementations differ by about as much as quantised and unquantised logits do.  The oracle shows this
by itself (its own logits move that much when its quantiser inputs are rounded to f16 first), so the end-to-end bar is
statistical: the CUDA path must be as close to the oracle as the oracle's f16-perturbed self is, must carry no more
quantisation noise against the unquantised oracle than the quantising oracle does, and must match row by row where
few codes flipped (the first layer's cache, which has passed one quantiser only)."""
import numpy as np
import pytest
import torch

from oracle import fdvlm_oracle as orc
from paper_2604_06832_b200 import inputs as I

pytestmark = pytest.mark.gpu

SMALL = I.ModelShape(n_layers=3, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, intermediate=1376, vocab=4096,
                     mask_id=4095, tie_embeddings=False, dtype=I.W8A8)


def B():
    from paper_2604_06832_b200 import binding
    return binding


@pytest.mark.parametrize("m,n,k", [(1, 128, 128), (8, 200, 688), (32, 2560, 2048), (33, 1000, 1376), (64, 4096, 512),
                                   (5, 72, 2048), (32, 2048, 11008), (48, 300, 3584)])
def test_op_linear_w8a8_quantises_like_the_oracle(m, n, k):
    g = torch.Generator().manual_seed(m * 1000 + n + k)
    x = torch.randn(m, k, generator=g) * torch.exp(2.0 * torch.randn(m, 1, generator=g))   # row magnitudes over ~3 decades
    if m >= 8:
        x[2] = 0.0                      # an all-zero row: scale 1, all codes 0
        x[3, k // 2] = 3000.0           # one outlier sets the row's scale; the rest falls to the bottom of the e4m3 range
    w = torch.randn(n, k, generator=g) * 0.05
    bias = torch.randn(n, generator=g) * 0.1
    xs = x.to(torch.bfloat16)
    # the operator stores its rows as f16 first (exact for all but the few bf16 values below f16's normal range), so
    # both sides quantise the same numbers
    xv = orc.to_f64(I.as_numpy_storage(xs)).astype(np.float16).astype(np.float64)
    ws, sc = I.quantize_e4m3_rows(w)
    wv = orc.to_f64(ws.numpy()) * sc.double().numpy()[:, None]
    ref = orc.quantize_rows_e4m3(xv) @ wv.T + bias.double().numpy()
    y = B().op_linear(xs.cuda(), ws.cuda(), sc.cuda(), bias.cuda(), dtype=B().DT_W8A8)
    torch.cuda.synchronize()
    got = y.double().cpu().numpy()
    row_scale = np.maximum(np.abs(ref).max(axis=1, keepdims=True), 1.0)
    err = (np.abs(got - ref) / row_scale).max()
    assert err <= 2e-4, err                                    # exact code products, fp32 accumulation
    # and the quantiser is really in the path: the unquantised product is visibly different
    plain = xv @ wv.T + bias.double().numpy()
    if k >= 128:
        assert (np.abs(plain - ref) / row_scale).max() > 2e-3


def test_op_linear_w8a8_rejects_unsupported_k():
    b = B()
    x = torch.zeros(4, 24, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(64, 24, dtype=torch.uint8, device="cuda")
    with pytest.raises(b.FdvlmError):
        b.op_linear(x, w, torch.ones(64, device="cuda"), None, dtype=b.DT_W8A8)


def _three_oracles(shape, w):
    """quantising oracle, unquantised oracle, and the quantising oracle with its quantiser inputs rounded to f16 first
    (a perturbation in the last bits, planted on the CPU side, that shows how far a correct implementation may drift)"""
    wn = I.weights_to_numpy(w)
    o8, o16 = orc.Oracle(shape, wn, act_fp8=True), orc.Oracle(shape, wn)
    o8p = orc.Oracle(shape, wn, act_fp8=True)
    plain_act = o8p._act
    o8p._act = lambda a: plain_act(np.asarray(a, dtype=np.float64).astype(np.float16).astype(np.float64))
    return o8, o16, o8p


def _rms(a):
    return float(np.sqrt(np.mean(np.square(a))))


@pytest.mark.parametrize("shape,B_,L_e,L_t", [(SMALL, 32, 33, 40),
                                              (SMALL.with_(n_q_heads=4, n_kv_heads=4, head_dim=64, hidden=384, intermediate=1120,
                                                           vocab=3000, mask_id=2999), 16, 20, 20),
                                              (SMALL.with_(tie_embeddings=True), 7, 5, 9),
                                              (SMALL.with_(n_layers=8), 32, 20, 20)])
def test_w8a8_model_is_as_close_to_the_oracle_as_rounding_allows(shape, B_, L_e, L_t):
    b = B()
    w = I.make_weights(shape, 7, gain_spread=0.5)        # generic norm gains: no activation sits on a rounding tie
    o8, o16, o8p = _three_oracles(shape, w)
    st = torch.cuda.Stream()
    h = b.Handle(shape, b.weights_to_device(w), max_seq=256, max_block=64, stream=st)
    emb, toks = I.make_prefix(shape, L_e, L_t, 3)
    for o in (o8, o16, o8p):
        o.prefill(I.as_numpy_storage(emb), toks.numpy(), want_logits=False)
        o.block_begin(B_)
    r8, r16, r8p = (o.block_step(orc.TOPK, 0.9, B_) for o in (o8, o16, o8p))
    lg = torch.empty(B_, shape.vocab, dtype=torch.float32, device="cuda")
    cf = torch.empty(B_, dtype=torch.float32, device="cuda")
    L = L_e + L_t
    with torch.cuda.stream(st):
        h.prefill(emb.cuda(), toks.cuda())
        h.block_begin(B_)
        h.block_step(b.RULE_TOPK, 0.9, B_, logits=lg, conf=cf)
        h.synchronize()
        k0 = h.cache_read(0, 0, 0, L).double().cpu().numpy()
        v0 = h.cache_read(0, 1, 0, L).double().cpu().numpy()
    h.close()
    g = lg.double().cpu().numpy()
    noise = r8["logits"] - r16["logits"]                  # what quantising the activations does to the logits
    drift = r8p["logits"] - r8["logits"]                  # what last-bit differences at the quantisers do to them
    d8, d16 = g - r8["logits"], g - r16["logits"]
    assert _rms(noise) > 1e-2                             # the quantiser matters here, or the bounds below say nothing
    assert _rms(d8) <= 1.25 * _rms(drift), (_rms(d8), _rms(drift))
    assert np.abs(d8).max() <= 1.5 * np.abs(drift).max(), (np.abs(d8).max(), np.abs(drift).max())
    assert _rms(d16) <= 1.15 * _rms(noise), (_rms(d16), _rms(noise))          # no more quantisation noise than the oracle's
    assert abs(float(np.mean(d8))) <= 0.1 * _rms(noise)                      # and no bias
    cerr = np.abs(cf.double().cpu().numpy() - r8["conf"])
    assert cerr.max() <= 1.5 * max(np.abs(r8p["conf"] - r8["conf"]).max(), 1e-3), cerr.max()
    # the first layer's K/V have passed ONE quantiser: few codes differ, each by one step, so the difference stays far
    # below what quantising does
    for got, ref, unq in ((k0, o8.K[0][:L], o16.K[0][:L]), (v0, o8.V[0][:L], o16.V[0][:L])):
        per_row = np.abs(got - ref).reshape(L, -1).max(axis=1)
        effect = np.abs(ref - unq).reshape(L, -1).max(axis=1)
        assert np.median(per_row) <= 0.25 * np.median(effect), (np.median(per_row), np.median(effect))
        assert _rms(got - ref) <= 0.35 * _rms(ref - unq), (_rms(got - ref), _rms(ref - unq))


def test_w8a8_give_up_path_and_recovery():
    """The quantising GEMM kind under the poison flag: every role (the converter warps included) leaves by the branch a
    timed-out wait takes, the call reports FDVLM_ERR_TIMEOUT, and after the flag is cleared the handle computes, bit for
    bit, what it computed before (the path is deterministic)."""
    b = B()
    w = I.make_weights(SMALL, 7, gain_spread=0.5)
    st = torch.cuda.Stream()
    h = b.Handle(SMALL, b.weights_to_device(w), max_seq=128, max_block=64, stream=st)
    emb, toks = I.make_prefix(SMALL, 10, 14, 3)
    lg = [torch.empty(16, SMALL.vocab, dtype=torch.float32, device="cuda") for _ in range(2)]
    with torch.cuda.stream(st):
        h.prefill(emb.cuda(), toks.cuda())
        h.block_begin(16)
        h.block_step(b.RULE_TOPK, 0.0, 4, logits=lg[0])
        h.synchronize()
        h.reset()
        h.debug_poison(True)
        h.prefill(emb.cuda(), toks.cuda())
        with pytest.raises(b.FdvlmError) as e:
            h.synchronize()
        assert e.value.code == b.ERR_TIMEOUT
        h.debug_poison(False)
        h.reset()
        h.prefill(emb.cuda(), toks.cuda())
        h.block_begin(16)
        h.block_step(b.RULE_TOPK, 0.0, 4, logits=lg[1])
        h.synchronize()
    assert torch.equal(lg[0], lg[1])
    h.close()
