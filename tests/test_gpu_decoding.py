"""GPU parity of the paper-convention decoding paths against the oracle, through the C ABI: denoise steps under
shift-by-one with an AR-seeded block (Sec. 3.4 "causal context decoding"), the verify commit that returns every row's
causal prediction, cache cropping, and whole iterations of linear self-speculative decoding (Appendix B, Alg. 1)."""
import numpy as np
import pytest
import torch

from oracle import fdvlm_oracle as orc
from paper_2604_06832_b200 import inputs as I
from tests.helpers import MARGIN, TOL, make_pair, upload_prefix

pytestmark = pytest.mark.gpu

SMALL_BF16 = I.ModelShape(n_layers=3, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, intermediate=1376,
                          vocab=4096, mask_id=4095, tie_embeddings=True, dtype=I.BF16)


def B():
    from paper_2604_06832_b200 import binding
    return binding


def both_prefill(oracle, handle, shape, ne, nt, seed):
    emb, toks = I.make_prefix(shape, ne, nt, seed)
    last_ref = oracle.prefill(I.as_numpy_storage(emb), toks.numpy())
    last = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
    handle.prefill(*upload_prefix(emb, toks), last)
    return last_ref, last


def sure_rows(logits, mask_id, gap=None):
    """Rows whose argmax is decided clearly: top-2 probability margin above 1e-3 (and, for the scaled-logit variants,
    a top-2 logit gap above `gap`, the logit error bound of the dtype)."""
    pred, conf, margin = orc.confidence(logits, mask_id)
    sure = margin > MARGIN
    if gap is not None:
        l = logits.copy()
        l[:, mask_id] = -np.inf
        top2 = np.sort(l, axis=1)[:, -2:]
        sure = sure & ((top2[:, 1] - top2[:, 0]) > gap)
    return pred, conf, sure


@pytest.mark.parametrize("shape,gain,B_,rule,tau,k", [(I.TINY, 16.0, 8, orc.THRESHOLD, 0.5, 0), (I.TINY, 16.0, 8, orc.TOPK, 0.0, 3),
                                                     (SMALL_BF16, 20.0, 16, orc.THRESHOLD, 0.6, 0), (SMALL_BF16, 1.0, 32, orc.TOPK, 0.0, 8)])
def test_shift_by_one_steps_match_oracle(shape, gain, B_, rule, tau, k):
    b = B()
    oracle, handle, _ = make_pair(shape, 21, max_seq=160, final_gain=gain)
    last_ref, _ = both_prefill(oracle, handle, shape, 20, 12, 5)
    seed = int(np.argmax(last_ref[:shape.mask_id]))
    tol = dict(TOL[shape.dtype])
    gap = None if gain == 1.0 else 2 * tol["logits"] * gain       # scaled logits: errors scale with the gain
    if gain != 1.0:
        # scaled-logit variant: logit errors scale with the gain, and a probability near 1/2 moves by a quarter of the
        # logit error (the same bounds as the other scaled-logit parity tests)
        tol["logits"] *= gain
        if shape.dtype != I.F32:
            tol["conf"] = 5e-2
    init = np.full(B_, shape.mask_id, dtype=np.int64)
    init[0] = seed
    oracle.block_begin(B_, init)
    handle.block_begin(B_, torch.from_numpy(init.astype(np.int32)).cuda())
    g_logits = torch.empty(B_, shape.vocab, dtype=torch.float32, device="cuda")
    g_conf = torch.empty(B_, dtype=torch.float32, device="cuda")
    g_pred = torch.empty(B_, dtype=torch.int32, device="cuda")
    g_um = torch.empty(B_, dtype=torch.uint8, device="cuda")
    g_tok = torch.empty(B_, dtype=torch.int32, device="cuda")
    code = b.RULE_THRESHOLD if rule == orc.THRESHOLD else b.RULE_TOPK
    steps = clear = 0
    while oracle.masked.any():
        handle.block_set_tokens(torch.from_numpy(oracle.block_tokens.astype(np.int32)).cuda())   # replay mode
        rec = oracle.block_step(rule, tau, k, pred_shift=1)
        info = handle.block_step(code, tau, k, logits=g_logits, conf=g_conf, pred=g_pred, unmask=g_um, block_tokens=g_tok,
                                 pred_shift=1)
        steps += 1
        assert np.abs(g_logits.double().cpu().numpy() - rec["logits"]).max() <= tol["logits"]
        m = rec["masked_before"]
        pos_conf_g = g_conf.double().cpu().numpy()[:-1]                 # position i + 1 takes row i
        assert np.abs(pos_conf_g - rec["pos_conf"][1:])[m[1:]].max() <= tol["conf"]
        um = g_um.cpu().numpy().astype(bool)
        assert not um[0] and not (um & ~m).any() and um.sum() >= 1 and info.n_unmasked == um.sum()
        _, _, sure_row = sure_rows(rec["logits"], shape.mask_id, gap)
        sure_pos = np.concatenate([[False], sure_row[:-1]])
        # selection decisions clear of the confidence tolerance?
        c = np.sort(rec["pos_conf"][m])[::-1]
        if rule == orc.THRESHOLD:
            ok = not np.any(np.abs(rec["pos_conf"][m] - tau) <= tol["conf"])
            if ok and not np.any(rec["pos_conf"][m] > tau):
                ok = c.size == 1 or (c[0] - c[1]) > 2 * tol["conf"]
        else:
            kk = min(k, c.size)
            ok = kk == c.size or (c[kk - 1] - c[kk]) > 2 * tol["conf"]
        if ok:
            clear += 1
            assert np.array_equal(um, rec["unmask"]) and info.n_remaining == rec["n_remaining"]
            toks = g_tok.cpu().numpy()
            good = ~um | sure_pos
            assert np.array_equal(toks[good], rec["block_tokens"][good])
    assert steps >= 1 and clear >= 1
    handle.block_set_tokens(torch.from_numpy(oracle.block_tokens.astype(np.int32)).cuda())
    # verify commit: every row's causal prediction
    d = oracle.block_tokens.copy()
    ref_all = oracle.commit_block(all_rows=True)
    a_ref, conf_ref, sure = sure_rows(ref_all, shape.mask_id, gap)
    row_pred = torch.empty(B_, dtype=torch.int32, device="cuda")
    row_conf = torch.empty(B_, dtype=torch.float32, device="cuda")
    nxt = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
    handle.commit_block_verify(row_pred, row_conf, nxt)
    assert handle.cache_len() == oracle.cache_len
    assert np.abs(nxt.double().cpu().numpy() - ref_all[-1]).max() <= tol["logits"]
    assert np.abs(row_conf.double().cpu().numpy() - conf_ref).max() <= tol["conf"]
    assert np.array_equal(row_pred.cpu().numpy()[sure], a_ref[sure])
    assert gain == 1.0 or sure.sum() >= 1          # (random-init confidences are ~1e-4: no clear row there)
    # crop, then re-commit a shorter block: caches agree again
    keep = oracle.cache_len - B_ + 3
    oracle.truncate(keep)
    handle.truncate(keep)
    assert handle.cache_len() == keep
    oracle.block_begin(2, d[3:5])
    handle.block_begin(2, torch.from_numpy(d[3:5].astype(np.int32)).cuda())
    oracle.commit_block()
    handle.commit_block()
    for layer in range(shape.n_layers):
        for which, ref in ((0, oracle.K[layer]), (1, oracle.V[layer])):
            got = handle.cache_read(layer, which, keep - 2, 4).double().cpu().numpy()
            assert np.abs(got - ref[keep - 2:keep + 2]).max() <= (1e-4 if shape.dtype == I.F32 else 2e-2)
    handle.close()


@pytest.mark.parametrize("shape,gain,B_", [(I.TINY, 16.0, 1), (I.TINY, 16.0, 4), (I.TINY, 16.0, 8), (SMALL_BF16, 24.0, 16)])
def test_self_speculative_iterations_match_oracle(shape, gain, B_):
    """Both sides run Alg. 1 from the same seed.  An iteration is compared when every argmax its outcome rests on is
    clear in the oracle: the draft rows that fill positions 1 .. k and the verify rows 0 .. k-1 (k = accepted length;
    later positions cannot change the outcome, the verify pass being causal).  The first unclear iteration ends the
    comparison, since the two caches may then legitimately differ."""
    oracle, handle, _ = make_pair(shape, 33, max_seq=256, final_gain=gain)
    last_ref, _ = both_prefill(oracle, handle, shape, 10, 14, 9)
    tol = TOL[shape.dtype]
    gap = 2 * tol["logits"] * gain
    seed = int(np.argmax(last_ref[:shape.mask_id]))
    draft = torch.empty(B_, dtype=torch.int32, device="cuda")
    a_dev = torch.empty(B_, dtype=torch.int32, device="cuda")
    compared = total_accepted = 0
    for _ in range(6):
        # the oracle's iteration, keeping the logits its decisions rest on
        L0 = oracle.cache_len
        init = np.full(B_, shape.mask_id, dtype=np.int64)
        init[0] = seed
        oracle.block_begin(B_, init)
        sure_draft = np.ones(B_, dtype=bool)
        if B_ > 1:
            rec = oracle.block_step(orc.THRESHOLD, -np.inf, 0, pred_shift=1)
            sure_draft = sure_rows(rec["logits"], shape.mask_id, gap)[2]
        d = oracle.block_tokens.copy()
        a, _, sure = sure_rows(oracle.commit_block(all_rows=True), shape.mask_id, gap)
        mism = [j for j in range(B_ - 1) if a[j] != d[j + 1]]
        k = (mism[0] if mism else B_ - 1) + 1
        clear = bool(sure_draft[:min(k, B_ - 1)].all()) and bool(sure[:k].all())
        oracle.truncate(L0 + k)
        info = handle.spec_block(B_, seed, draft, a_dev)
        assert 1 <= info.accepted <= B_ and info.cache_len == handle.cache_len()
        if not clear:
            break
        compared += 1
        total_accepted += k
        n_d = min(k + 1, B_)
        assert np.array_equal(draft.cpu().numpy()[:n_d], d[:n_d])
        assert np.array_equal(a_dev.cpu().numpy()[:k], a[:k])
        assert info.accepted == k and info.next_token == int(a[k - 1]) and info.cache_len == oracle.cache_len
        seed = int(a[k - 1])
    assert compared >= (2 if shape.dtype == I.F32 else 1) and total_accepted >= compared
    handle.close()


def test_speculative_decoding_on_the_gpu_is_lossless():
    # the accepted tokens of block size 8 are the greedy chain that block size 1 (plain autoregression) produces
    shape = I.TINY
    outs = []
    for B_ in (1, 8):
        _, handle, _ = make_pair(shape, 33, max_seq=256, final_gain=16.0)
        emb, toks = I.make_prefix(shape, 10, 14, 9)
        last = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
        handle.prefill(*upload_prefix(emb, toks), last)
        l = last.cpu().numpy()
        l[shape.mask_id] = -np.inf
        seq = [int(np.argmax(l))]
        a_dev = torch.empty(B_, dtype=torch.int32, device="cuda")
        while len(seq) < 24:
            info = handle.spec_block(B_, seq[-1], None, a_dev)
            seq.extend(int(t) for t in a_dev.cpu().numpy()[:info.accepted])
            assert seq[-1] == info.next_token and handle.cache_len() == 24 + len(seq) - 1
        outs.append(seq[:24])
        handle.close()
    assert outs[0] == outs[1]


@pytest.mark.parametrize("shift", [0, 1])
def test_topk_block_decode_without_host_round_trips_equals_stepwise(shift):
    b = B()
    shape, Bsz, k = I.TINY, 8, 3
    _, handle, _ = make_pair(shape, 4, max_seq=128, final_gain=16.0)
    toks = I.random_tokens(shape, 30, 2).cuda()
    init = torch.full((Bsz,), shape.mask_id, dtype=torch.int32, device="cuda")
    if shift:
        init[0] = 77
    out = []
    for mode in ("stepwise", "fused"):
        handle.reset()
        handle.prefill(None, toks)
        got = torch.empty(Bsz, dtype=torch.int32, device="cuda")
        if mode == "stepwise":
            handle.block_begin(Bsz, init)
            n = 0
            while True:
                info = handle.block_step(b.RULE_TOPK, 0.0, k, block_tokens=got, pred_shift=shift)
                n += 1
                if info.n_remaining == 0:
                    break
        else:
            info = handle.decode_block_topk(Bsz, k, init, shift, got)
            n = info.step_index
        assert info.n_remaining == 0 and n == -(-(Bsz - shift) // k)
        nxt = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
        handle.commit_block(nxt)
        out.append((got.cpu().numpy().copy(), nxt.cpu().numpy().copy(), n))
    assert np.array_equal(out[0][0], out[1][0]) and np.array_equal(out[0][1], out[1][1]) and out[0][2] == out[1][2]
    assert (out[1][0] != shape.mask_id).all()
    # shift-by-one needs a given first position
    handle.reset()
    handle.prefill(None, toks)
    with pytest.raises(b.FdvlmError) as e:
        handle.decode_block_topk(Bsz, k, None, 1)
    assert e.value.code == b.ERR_STATE
    handle.close()


def test_decoding_entry_point_errors():
    b = B()
    _, handle, _ = make_pair(I.TINY, 0, max_seq=64, max_block=8)
    toks = I.random_tokens(I.TINY, 20, 2).cuda()
    handle.prefill(None, toks)
    handle.block_begin(4)                                   # position 0 masked: shift-by-one cannot start
    with pytest.raises(b.FdvlmError) as e:
        handle.block_step(b.RULE_THRESHOLD, 0.9, pred_shift=1)
    assert e.value.code == b.ERR_STATE
    with pytest.raises(b.FdvlmError) as e:
        handle.block_step(b.RULE_THRESHOLD, 0.9, pred_shift=2)
    assert e.value.code == b.ERR_INVALID_ARG
    with pytest.raises(b.FdvlmError) as e:
        handle.truncate(10)                                 # inside an open block
    assert e.value.code == b.ERR_STATE
    handle.block_step(b.RULE_THRESHOLD, -1.0)
    handle.commit_block()
    with pytest.raises(b.FdvlmError) as e:
        handle.truncate(25)
    assert e.value.code == b.ERR_INVALID_ARG
    with pytest.raises(b.FdvlmError) as e:
        handle.spec_block(4, I.TINY.mask_id)
    assert e.value.code == b.ERR_INVALID_ARG
    with pytest.raises(b.FdvlmError) as e:
        handle.spec_block(9, 5)
    assert e.value.code == b.ERR_CAPACITY
    handle.truncate(0)
    assert handle.cache_len() == 0
    handle.close()
