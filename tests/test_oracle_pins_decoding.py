"""Pins for the oracle's paper-convention decoding (shift-by-one with an AR-seeded block, Sec. 3.4 "causal context
decoding") and its linear self-speculative iteration (Appendix B, Alg. 1).  What fixes them from outside: verification
by the causal pass makes speculative decoding lossless, so its output must be the greedy autoregressive chain computed
from scratch with the brute-force dense-mask routine; block size one is plain autoregression; reveal-all and tau = 1
schedules have closed-form step counts; the cropped cache must equal the cache of a dense causal pass."""
import numpy as np
import pytest

from oracle import fdvlm_oracle as orc
from paper_2604_06832_b200 import inputs as I

MICRO = I.ModelShape(n_layers=2, hidden=32, n_q_heads=4, n_kv_heads=2, head_dim=8, intermediate=48,
                     vocab=64, mask_id=63, tie_embeddings=True, dtype=I.F32)


def make(seed=3, std=0.3, **kw):
    w = I.make_weights(MICRO, seed, std=std, **kw)
    return orc.Oracle(MICRO, I.weights_to_numpy(w))


def greedy_chain(o, x_prefix, n_new):
    """Greedy AR continuation by full recomputation with an explicit causal mask (no cache, no blocks)."""
    x, out = x_prefix, []
    for _ in range(n_new):
        row = o.forward_dense(x, orc.causal_mask(len(x)))[-1]
        tok = int(np.argmax(row[:MICRO.mask_id]))
        out.append(tok)
        x = np.concatenate([x, o.embed_tokens([tok])], 0)
    return out


def start(o, ne=2, nt=5, seed=7):
    e, t = I.make_prefix(MICRO, ne, nt, seed)
    emb, toks = I.as_numpy_storage(e), t.numpy()
    last = o.prefill(emb, toks)
    x_prefix = np.concatenate([orc.to_f64(emb), o.embed_tokens(toks)], 0)
    return x_prefix, int(np.argmax(last[:MICRO.mask_id]))


@pytest.mark.parametrize("B", [1, 2, 3, 5, 8])
@pytest.mark.parametrize("gain", [1.0, 12.0])
def test_self_speculative_decoding_is_lossless(B, gain):
    # whatever the draft proposes, the accepted tokens are causal argmaxes given a verified prefix: the generated
    # sequence is the greedy chain, and every iteration accepts between 1 and B tokens
    o = make(final_gain=gain)
    x_prefix, seed = start(o)
    want = greedy_chain(o, x_prefix, 14)
    got, L0 = [seed], o.cache_len
    while len(got) < 14:
        rec = o.spec_block(B, got[-1])
        assert 1 <= rec["accepted"] <= B and len(rec["new_tokens"]) == rec["accepted"]
        assert rec["next_token"] == rec["new_tokens"][-1]
        got.extend(int(t) for t in rec["new_tokens"])
        assert o.cache_len == L0 + len(got) - 1          # everything but the newest token is committed
    assert got[:14] == want


def test_accept_rule_on_a_forced_mismatch_and_cache_crop():
    # draft rows replaced by hand: agreement on the first two drafted positions, disagreement on the third
    o = make()
    x_prefix, seed = start(o)
    chain = greedy_chain(o, x_prefix, 6)                  # chain[0] == seed
    assert chain[0] == seed
    B, L0 = 5, o.cache_len
    wrong = (chain[3] + 1) % MICRO.mask_id
    d = np.array([chain[0], chain[1], chain[2], wrong, chain[4]])
    o.block_begin(B, d)
    a = orc.confidence(o.commit_block(all_rows=True), MICRO.mask_id)[0]
    assert list(a[:3]) == chain[1:4]                      # a_j continues the verified prefix
    mism = [j for j in range(B - 1) if a[j] != d[j + 1]]
    assert mism[0] == 2                                   # a_2 = chain[3] != wrong
    o.truncate(L0 + 3)
    # the cropped cache is the cache of the dense causal pass over prefix + d_0..d_2
    x = np.concatenate([x_prefix, o.embed_tokens(d[:3])], 0)
    o3 = make()
    e, t = I.make_prefix(MICRO, 2, 5, 7)
    o3.prefill(I.as_numpy_storage(e), t.numpy())
    o3.block_begin(3, d[:3])
    o3.commit_block()
    for l in range(MICRO.n_layers):
        assert np.abs(o.K[l] - o3.K[l]).max() < 1e-12 and np.abs(o.V[l] - o3.V[l]).max() < 1e-12
    assert o.cache_len == o3.cache_len == len(x)


def test_seeded_block_size_one_is_plain_autoregression():
    o = make()
    x_prefix, seed = start(o)
    want = greedy_chain(o, x_prefix, 6)
    got = [seed]
    for _ in range(5):
        toks, steps, nxt = o.decode_block_seeded(1, got[-1], orc.THRESHOLD, 0.9)
        assert steps == [] and list(toks) == [got[-1]]
        got.append(nxt)
    assert got == want


def test_shift_by_one_reveal_all_takes_row_i_minus_1():
    o = make(final_gain=8.0)
    _, seed = start(o)
    B = 6
    init = np.full(B, MICRO.mask_id)
    init[0] = seed
    o.block_begin(B, init)
    logits = o.block_forward()
    rec = o.block_step(orc.THRESHOLD, -1.0, 0, pred_shift=1)
    assert rec["n_remaining"] == 0 and rec["n_unmasked"] == B - 1
    for i in range(1, B):
        assert rec["block_tokens"][i] == int(np.argmax(logits[i - 1][:MICRO.mask_id]))
    assert rec["block_tokens"][0] == seed and not rec["unmask"][0]


@pytest.mark.parametrize("rule,tau,k,B,expect", [(orc.THRESHOLD, 1.0, 0, 6, 5), (orc.THRESHOLD, -1.0, 0, 6, 1),
                                                 (orc.TOPK, 0.0, 2, 7, 3), (orc.TOPK, 0.0, 8, 5, 1)])
def test_seeded_decode_step_counts(rule, tau, k, B, expect):
    # B - 1 masked positions: one per step at tau = 1 (Sec. 4.5), all at once below any confidence, ceil((B-1)/k) for top-k
    o = make()
    _, seed = start(o)
    toks, steps, nxt = o.decode_block_seeded(B, seed, rule, tau, k)
    assert len(steps) == expect and toks[0] == seed and MICRO.mask_id not in toks and 0 <= nxt < MICRO.mask_id
    assert sum(s["n_unmasked"] for s in steps) == B - 1


def test_shift_needs_a_given_first_position():
    o = make()
    start(o)
    o.block_begin(4)
    with pytest.raises(AssertionError):
        o.block_step(orc.THRESHOLD, 0.9, 0, pred_shift=1)


def test_planted_off_by_one_in_crop_is_caught(monkeypatch):
    # keeping one cache entry too many (the rejected draft token's) must break losslessness: the pin above would fail
    o = make()
    x_prefix, seed = start(o)
    want = greedy_chain(o, x_prefix, 12)
    good = orc.Oracle.truncate

    def bad(self, new_len):
        good(self, min(new_len + 1, self.cache_len))
    monkeypatch.setattr(orc.Oracle, "truncate", bad)
    got, partial = [seed], False
    while len(got) < 12:
        rec = o.spec_block(4, got[-1])
        partial = partial or rec["accepted"] < 4
        got.extend(int(t) for t in rec["new_tokens"])
    assert partial and got[:12] != want


def test_golden_masks_and_accept_rule_of_algorithm_1():
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "alg1_masks_and_accept.txt")
    lines = [l.strip() for l in open(path) if l.strip() and not l.startswith("#")]
    i = n_accept = 0
    while i < len(lines):
        parts = lines[i].split()
        if parts[0] in ("draft_mask", "verify_mask"):
            L, B_ = int(parts[1]), int(parts[2])
            want = np.array([[int(x) for x in lines[i + 1 + r].split()] for r in range(B_)], dtype=bool)
            got = orc.draft_mask(L, B_)[L:] if parts[0] == "draft_mask" else orc.verify_mask(L, B_)
            assert got.shape == want.shape and np.array_equal(got, want)
            i += 1 + B_
        else:
            assert parts[0] == "accept"
            d, a, k, new = [[int(x) for x in f.split()] for f in lines[i][len("accept"):].split("|")]
            assert orc.accept_length(np.array(a), np.array(d)) == k[0] and a[:k[0]] == new
            n_accept += 1
            i += 1
    assert n_accept == 5
