"""Pins for the oracle's quadratic self-speculative decoding (Appendix B, Alg. 2).  What fixes it from outside: the input
layout, position ids, mask and accept loop worked by hand from the printed rules (tests/golden/); the cached forward
against the brute-force dense-mask routine over the whole sequence; the first tokens of the groups, which by rule (b)
are exactly a causal pass over the draft; group 0, which is an ordinary denoise block; the kept cache entries, which
must be those of a causal pass over the accepted tokens; and, over a whole decode, every verified token must be the
greedy continuation of what precedes it."""
import os

import numpy as np
import pytest

from oracle import fdvlm_oracle as orc
from paper_2604_06832_b200 import inputs as I

MICRO = I.ModelShape(n_layers=2, hidden=32, n_q_heads=4, n_kv_heads=2, head_dim=8, intermediate=48,
                     vocab=64, mask_id=63, tie_embeddings=True, dtype=I.F32)
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "alg2_quadratic_mask_positions_accept.txt")


def make(seed=3, std=0.3, **kw):
    w = I.make_weights(MICRO, seed, std=std, **kw)
    return orc.Oracle(MICRO, I.weights_to_numpy(w))


def start(o, ne=2, nt=4, seed=7):
    e, t = I.make_prefix(MICRO, ne, nt, seed)
    emb, toks = I.as_numpy_storage(e), t.numpy()
    last = o.prefill(emb, toks)
    return np.concatenate([orc.to_f64(emb), o.embed_tokens(toks)], 0), last


def _ints(text):
    return [int(t) for t in text.split()]


def test_golden_layout_positions_mask_and_accept_loop_of_algorithm_2():
    lines = [l.strip() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    i, seen = 0, set()
    while i < len(lines):
        kind, _, rest = lines[i].partition(" ")
        seen.add(kind)
        if kind == "input":
            B, d, q = rest.split("|")
            want = np.array(_ints(q))
            got = orc.quad_input(_ints(d), MICRO.mask_id)
            assert np.array_equal(np.where(got == MICRO.mask_id, -1, got), want) and len(got) == int(B) * (int(B) + 1)
            i += 1
        elif kind == "positions":
            head, pos = rest.split("|")
            s, B = _ints(head)
            assert orc.quad_positions(s, B).tolist() == _ints(pos)
            i += 1
        elif kind in ("mask", "mask_chain"):
            B = int(rest)
            n = B * (B + 1)
            want = np.array([_ints(l) for l in lines[i + 1:i + 1 + n]], dtype=bool)
            assert want.shape == (n, n)
            assert np.array_equal(orc.quad_mask(B, chain=(kind == "mask_chain")), want)
            i += 1 + n
        elif kind == "accept":
            d, P, k, nxt = rest.split("|")
            P = np.array([_ints(r) for r in P.split(";")])
            got_k, got_next = orc.quad_accept(P, _ints(d))
            assert got_k == int(k) and got_next.tolist() == _ints(nxt)
            i += 1
        else:
            raise AssertionError(lines[i])
    assert seen == {"input", "positions", "mask", "mask_chain", "accept"}


def _dense_quad_logits(o, x_prefix, d, chain):
    """the B(B+1) rows recomputed from scratch: [prefix ; q] under one explicit mask, prefix rows causal"""
    B, L = len(d), len(x_prefix)
    n = B * (B + 1)
    allowed = np.zeros((L + n, L + n), dtype=bool)
    allowed[:L, :L] = orc.causal_mask(L)
    allowed[L:, :L] = True                                   # rule (a)
    allowed[L:, L:] = orc.quad_mask(B, chain)
    pos = np.concatenate([np.arange(L), orc.quad_positions(L, B)])
    x = np.concatenate([x_prefix, o.embed_tokens(orc.quad_input(d, MICRO.mask_id))], 0)
    return o.forward_dense(x, allowed, pos)[L:]


@pytest.mark.parametrize("B,chain", [(1, False), (2, False), (3, False), (3, True)])
def test_cached_quadratic_forward_equals_the_brute_force_dense_mask(B, chain):
    o = make()
    x_prefix, _ = start(o)
    d = np.array([5, 17, 40][:B])
    want = _dense_quad_logits(o, x_prefix, d, chain)
    rec = o.quad_step(d, chain=chain)
    assert np.abs(rec["logits"] - want).max() < 1e-9


@pytest.mark.parametrize("chain", [False, True])
def test_first_tokens_are_a_causal_pass_and_group_zero_is_a_denoise_block(chain):
    B = 4
    d = np.array([5, 17, 40, 8])
    a, b, c = make(), make(), make()
    for o in (a, b, c):
        start(o)
    rec = a.quad_step(d, chain=chain)
    # rule (b): the first tokens read the cache and the first tokens before them -- Alg. 1's verify pass over d
    b.block_begin(B, d)
    causal = b.commit_block(all_rows=True)
    assert np.abs(rec["logits"][::B + 1] - causal).max() < 1e-9
    # rule (c) for group 0 -- except its first token, whose row is causal: an ordinary denoise pass over [d_0, M^B]
    # gives the same K / V for d_0 only in the first layer, so compare what must agree exactly: a one-layer model
    one = I.ModelShape(**{**MICRO.__dict__, "n_layers": 1})
    w = I.weights_to_numpy(I.make_weights(one, 3, std=0.3))
    o1, o2 = orc.Oracle(one, w), orc.Oracle(one, w)
    e, t = I.make_prefix(one, 2, 4, 7)
    for o in (o1, o2):
        o.prefill(I.as_numpy_storage(e), t.numpy())
    r1 = o1.quad_step(d, chain=chain)
    o2.block_begin(B + 1, np.concatenate([[d[0]], np.full(B, one.mask_id)]))
    assert np.abs(r1["logits"][1:B + 1] - o2.block_forward()[1:]).max() < 1e-9


def _greedy_draft(B, gain):
    """[seed, then the greedy continuation token by token] by one-token causal commits: a draft that verifies fully"""
    g = make(final_gain=gain)
    _, last = start(g)
    d = [int(np.argmax(last[:MICRO.mask_id]))]
    while len(d) < B:
        g.block_begin(1, [d[-1]])
        d.append(int(np.argmax(g.commit_block()[:MICRO.mask_id])))
    return np.array(d)


@pytest.mark.parametrize("gain", [1.0, 12.0])
@pytest.mark.parametrize("n_good", [1, 2, 3])
def test_kept_cache_entries_are_those_of_a_causal_pass_over_the_accepted_tokens(gain, n_good):
    # the draft follows the greedy chain for n_good tokens and then leaves it: exactly n_good are accepted
    B = 3
    a, b = make(final_gain=gain), make(final_gain=gain)
    start(a)
    start(b)
    d = _greedy_draft(B, gain)
    for j in range(n_good, B):
        d[j] = (d[j] + 1 + j) % MICRO.mask_id                # any other token
    L = a.cache_len
    rec = a.quad_step(d)
    k = rec["accepted"]
    assert k == n_good and a.cache_len == L + k and rec["new_tokens"].tolist() == d[:k].tolist()
    assert rec["next_draft"].tolist() == rec["P"][k - 1, 1:].tolist()
    b.block_begin(k, d[:k])
    b.commit_block(want_logits=False)
    for l in range(MICRO.n_layers):
        assert np.abs(a.K[l] - b.K[l]).max() < 1e-12 and np.abs(a.V[l] - b.V[l]).max() < 1e-12


def test_first_draft_equals_the_one_shot_pass_of_step_1():
    # Alg. 2 step 1 as printed: [prompt ; M^B] in ONE pass, prompt rows causal, mask rows reading everything;
    # d_i = argmax h_{L-1+i}
    o = make(final_gain=12.0)
    x_prefix, last = start(o)
    B, L = 4, len(x_prefix)
    x = np.concatenate([x_prefix, o.embed_tokens(np.full(B, MICRO.mask_id))], 0)
    dense = o.forward_dense(x, orc.draft_mask(L, B))
    want = [int(np.argmax(dense[L - 1 + i][:MICRO.mask_id])) for i in range(B)]
    assert o.quad_first_draft(B, last).tolist() == want and o.cache_len == L


@pytest.mark.parametrize("B", [1, 2, 3, 5])
@pytest.mark.parametrize("gain,chain", [(1.0, False), (12.0, False), (12.0, True)])
def test_whole_decode_every_verified_token_is_the_greedy_continuation(B, gain, chain):
    o = make(final_gain=gain)
    x_prefix, last = start(o)
    L0 = o.cache_len
    d = o.quad_first_draft(B, last)
    seq, verified = [], []
    for _ in range(6):
        rec = o.quad_step(d, chain=chain)
        k = rec["accepted"]
        assert 1 <= k <= B and len(rec["next_draft"]) == B
        seq.extend(int(t) for t in rec["new_tokens"])
        verified.extend([False] + [True] * (k - 1))         # d_0 of a block is taken as proposed, d_1.. were checked
        assert o.cache_len == L0 + len(seq)
        d = rec["next_draft"]
    # one dense causal pass over everything generated: its row p-1 is the autoregressive distribution of position p
    x = np.concatenate([x_prefix, o.embed_tokens(seq)], 0)
    dense = o.forward_dense(x, orc.causal_mask(len(x)))
    for p, (tok, ver) in enumerate(zip(seq, verified)):
        if ver:
            assert tok == int(np.argmax(dense[L0 + p - 1][:MICRO.mask_id])), p
    assert verified[0] is False and int(np.argmax(last[:MICRO.mask_id])) == seq[0]     # the very first token is the AR seed
    # and the cache is the cache of that causal pass
    fresh = make(final_gain=gain)
    fresh.forward_rows(x, orc.CAUSAL, update_cache=True)
    for l in range(MICRO.n_layers):
        assert np.abs(o.K[l] - fresh.K[l]).max() < 1e-9


def test_planted_errors_fail_the_pins(monkeypatch):
    good_pos, good_mask = orc.quad_positions, orc.quad_mask
    # position ids without the group offset
    monkeypatch.setattr(orc, "quad_positions", lambda s, B: np.array([s + j for _ in range(B) for j in range(B + 1)]))
    with pytest.raises(AssertionError):
        test_first_tokens_are_a_causal_pass_and_group_zero_is_a_denoise_block(False)
    with pytest.raises(AssertionError):
        test_golden_layout_positions_mask_and_accept_loop_of_algorithm_2()
    monkeypatch.setattr(orc, "quad_positions", good_pos)
    # first tokens reading every group's first token (no causality among them)
    def leaky(B, chain=False):
        m = good_mask(B, chain)
        m[::B + 1, ::B + 1] = True
        return m
    monkeypatch.setattr(orc, "quad_mask", leaky)
    with pytest.raises(AssertionError):
        test_first_tokens_are_a_causal_pass_and_group_zero_is_a_denoise_block(False)
    with pytest.raises(AssertionError):
        test_golden_layout_positions_mask_and_accept_loop_of_algorithm_2()
    monkeypatch.setattr(orc, "quad_mask", good_mask)
    # keeping the K / V of consecutive entries instead of every (B+1)-th
    good_append = orc.Oracle.append_cache
    monkeypatch.setattr(orc.Oracle, "append_cache", lambda self, k, v, rows: good_append(self, k, v, np.arange(len(rows))))
    with pytest.raises(AssertionError):
        test_kept_cache_entries_are_those_of_a_causal_pass_over_the_accepted_tokens(12.0, 3)
