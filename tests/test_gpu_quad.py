"""GPU parity of quadratic self-speculative decoding (Appendix B, Alg. 2) through the C ABI: the B (B+1)-row forward
under the group mask and the per-group position ids, the verify loop, the next draft and the kept cache entries, against
the oracle on the same seeded inputs.  The library orders the rows first tokens first (see the header); the oracle
keeps the paper's order, group after group: the tests permute.  Both sides are handed the same draft before every
iteration (replay), so one low-margin token cannot send them down different paths."""
import numpy as np
import pytest
import torch

from oracle import fdvlm_oracle as orc
from paper_2604_06832_b200 import inputs as I

from helpers import TOL, make_pair, upload_prefix

pytestmark = pytest.mark.gpu

TINY = I.TINY
SMALL_BF16 = I.ModelShape(n_layers=3, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, intermediate=1376,
                          vocab=4096, mask_id=4095, tie_embeddings=True, dtype=I.BF16)
SMALL_FP8 = SMALL_BF16.with_(dtype=I.FP8, tie_embeddings=False, n_q_heads=4, n_kv_heads=4, head_dim=64, hidden=384,
                             intermediate=1120, vocab=3000, mask_id=2999)
MARGIN = 1e-3


def B_():
    from paper_2604_06832_b200 import binding
    return binding


def to_paper_order(B):
    """index array p with paper_rows = library_rows[p]: paper row i (B+1) + j  <-  library row i (j = 0) or B + i B + j - 1"""
    return np.array([i if j == 0 else B + i * B + j - 1 for i in range(B) for j in range(B + 1)])


def run_iterations(shape, B, chain, n_iter, stream, final_gain=1.0, L_e=5, L_t=9, tol=None):
    b = B_()
    tol = tol or TOL[shape.dtype]
    st = torch.cuda.Stream() if stream else None
    oracle, handle, _ = make_pair(shape, 11, max_seq=256, max_block=64, stream=st, final_gain=final_gain)
    emb, toks = I.make_prefix(shape, L_e, L_t, 3)
    last = oracle.prefill(I.as_numpy_storage(emb), toks.numpy())
    n = B * (B + 1)
    perm = to_paper_order(B)
    g_last = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
    g_draft = torch.empty(B, dtype=torch.int32, device="cuda")
    g_acc = torch.empty(B, dtype=torch.int32, device="cuda")
    g_next = torch.empty(B, dtype=torch.int32, device="cuda")
    g_pred = torch.empty(n, dtype=torch.int32, device="cuda")
    g_logits = torch.empty(n, shape.vocab, dtype=torch.float32, device="cuda")
    stats = dict(logit_err=0.0, sure_rows=0, clear_iters=0, accepted=[])
    ctx = torch.cuda.stream(st) if st is not None else torch.cuda.stream(torch.cuda.current_stream())
    with ctx:
        e, t = upload_prefix(emb, toks)
        handle.prefill(e, t, g_last)
        handle.synchronize()
        assert np.abs(g_last.double().cpu().numpy() - last).max() <= tol["logits"]
        d = oracle.quad_first_draft(B, last)
        handle.quad_begin(B, int(d[0]), chain=chain, draft=g_draft)
        handle.synchronize()
        # step 1: the first token is given, the others come from mask rows: compare where the oracle's margin is clear
        x = oracle.embed_tokens(np.full(B, shape.mask_id, dtype=np.int64))
        m1 = orc.confidence(oracle.logits_of(oracle.forward_rows(x, orc.BIDIR, False)), shape.mask_id)[2]
        gd = g_draft.cpu().numpy()
        assert gd[0] == d[0]
        sure1 = np.concatenate([[True], m1[:B - 1] > MARGIN])
        assert np.array_equal(gd[sure1], d[sure1])
        assert handle.cache_len() == oracle.cache_len
        for _ in range(n_iter):
            handle.quad_set_draft(torch.from_numpy(d.astype(np.int32)).cuda())
            L0 = oracle.cache_len
            rec = oracle.quad_step(d, chain=chain)
            info = handle.quad_step(accepted_tokens=g_acc, next_draft=g_next, row_pred=g_pred, logits=g_logits)
            got = g_logits.double().cpu().numpy()[perm]
            err = np.abs(got - rec["logits"]).max()
            stats["logit_err"] = max(stats["logit_err"], float(err))
            assert err <= tol["logits"], f"logits max-abs err {err}"
            margin = orc.confidence(rec["logits"], shape.mask_id)[2].reshape(B, B + 1)
            pred = g_pred.cpu().numpy()[perm].reshape(B, B + 1)
            sure = margin > MARGIN
            stats["sure_rows"] += int(sure.sum())
            assert np.array_equal(pred[sure], rec["P"][sure]), "predictions differ where the top-2 margin is clear"
            k = rec["accepted"]
            # the kernel's loop against Alg. 2's loop run on the kernel's OWN predictions: always comparable
            own_k, own_next = orc.quad_accept(pred, d)
            acc, nxt = g_acc.cpu().numpy(), g_next.cpu().numpy()
            assert info.accepted == own_k and info.cache_len == L0 + own_k == handle.cache_len()
            assert np.array_equal(acc[:own_k], d[:own_k]) and (acc[own_k:] == -1).all() and np.array_equal(nxt, own_next)
            # against the oracle where the verify loop's reads, P_{0,0} .. P_{min(k, B-1)-1, 0}, are clear of the margin
            if sure[:min(k, B - 1), 0].all():
                stats["clear_iters"] += 1
                assert info.accepted == k and info.cache_len == oracle.cache_len
                ok = sure[k - 1, 1:]
                assert np.array_equal(nxt[ok], rec["next_draft"][ok])
                # kept cache entries: the first tokens of the accepted groups, at the positions they were accepted to
                for l in (0, shape.n_layers - 1):
                    for which, ref in ((0, oracle.K[l]), (1, oracle.V[l])):
                        gk = handle.cache_read(l, which, L0, k).double().cpu().numpy()
                        cerr = np.abs(gk - ref[L0:L0 + k]).max()
                        assert cerr <= max(tol["logits"], 2e-2 * np.abs(ref[L0:L0 + k]).max()), cerr
            elif info.accepted != k:
                break                                        # the two sides took different branches inside the margin
            stats["accepted"].append(k)
            d = rec["next_draft"]
        handle.quad_end()
    handle.close()
    return stats


@pytest.mark.parametrize("B", [1, 2, 3, 5, 7])
@pytest.mark.parametrize("chain", [False, True])
def test_quad_tiny_fp32(B, chain):
    stats = run_iterations(TINY, B, chain, n_iter=3, stream=False)
    assert stats["logit_err"] <= 1e-4


@pytest.mark.parametrize("shape", [SMALL_BF16, SMALL_FP8], ids=["bf16", "fp8"])
@pytest.mark.parametrize("B,chain", [(2, False), (4, False), (7, False), (5, True)])
def test_quad_small_tensor_core_path_on_a_stream(shape, B, chain):
    run_iterations(shape, B, chain, n_iter=2, stream=True)


def test_quad_peaked_model_decisions_are_compared():
    # confidences spread over (0, 1): most margins are clear, so predictions, accepted lengths and next drafts are compared
    stats = run_iterations(SMALL_BF16, 5, False, n_iter=3, stream=True, final_gain=16.0)    # at the stated bf16 bounds
    assert stats["sure_rows"] > 30 and stats["clear_iters"] == 3


def test_quad_fully_verifying_draft_is_accepted_whole():
    # a draft that IS the greedy chain must be accepted to the last token, and the cache must gain its K / V
    b = B_()
    shape, B = TINY, 4
    oracle, handle, w = make_pair(shape, 11, max_seq=256, max_block=64, final_gain=16.0)
    scratch = orc.Oracle(shape, I.weights_to_numpy(w))
    emb, toks = I.make_prefix(shape, 5, 9, 3)
    last = oracle.prefill(I.as_numpy_storage(emb), toks.numpy())
    d = [int(orc.confidence(scratch.prefill(I.as_numpy_storage(emb), toks.numpy())[None, :], shape.mask_id)[0][0])]
    while len(d) < B:
        scratch.block_begin(1, [d[-1]])
        d.append(int(orc.confidence(scratch.commit_block()[None, :], shape.mask_id)[0][0]))
    d = np.array(d)
    e, t = upload_prefix(emb, toks)
    handle.prefill(e, t)
    handle.quad_begin(B, int(d[0]))
    handle.quad_set_draft(torch.from_numpy(d.astype(np.int32)).cuda())
    L0 = oracle.cache_len
    rec = oracle.quad_step(d)
    info = handle.quad_step()
    assert rec["accepted"] == B and info.accepted == B and info.cache_len == L0 + B
    for l in range(shape.n_layers):
        gk = handle.cache_read(l, 0, L0, B).double().cpu().numpy()
        assert np.abs(gk - oracle.K[l][L0:]).max() <= 1e-4
    handle.close()


def test_quad_state_and_capacity_errors():
    b = B_()
    _, handle, _ = make_pair(TINY, 1, max_seq=128, max_block=64)
    with pytest.raises(b.FdvlmError):
        handle.quad_step()                                   # nothing open
    with pytest.raises(b.FdvlmError):
        handle.quad_begin(8, 3)                              # 72 rows
    with pytest.raises(b.FdvlmError):
        handle.quad_begin(3, TINY.mask_id)                   # the mask token is not a token
    handle.block_begin(4)
    with pytest.raises(b.FdvlmError):
        handle.quad_begin(3, 3)                              # inside an open block
    handle.close()
    _, small, _ = make_pair(TINY, 1, max_seq=128, max_block=16)
    with pytest.raises(b.FdvlmError):
        small.quad_begin(4, 3)                               # 20 rows > max_block
    small.close()
