"""GPU parity of the fused forward that commits a finished block and runs the next block's first denoise step (Sec. 3.3's
three masks in one pass): against the oracle, which makes the three calls one after the other."""
import numpy as np
import pytest
import torch

from oracle import fdvlm_oracle as orc
from paper_2604_06832_b200 import inputs as I

from helpers import TOL, compare_step, make_pair, upload_prefix

pytestmark = pytest.mark.gpu

SMALL_BF16 = I.ModelShape(n_layers=3, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, intermediate=1376,
                          vocab=4096, mask_id=4095, tie_embeddings=True, dtype=I.BF16)
SMALL_FP8 = SMALL_BF16.with_(dtype=I.FP8, tie_embeddings=False, n_q_heads=4, n_kv_heads=4, head_dim=64, hidden=384,
                             intermediate=1120, vocab=3000, mask_id=2999)


def B_():
    from paper_2604_06832_b200 import binding
    return binding


@pytest.mark.parametrize("shape,stream", [(I.TINY, False), (SMALL_BF16, True), (SMALL_FP8, True), (SMALL_BF16, False)],
                         ids=["tiny-f32", "bf16-graphs", "fp8-graphs", "bf16-launches"])
@pytest.mark.parametrize("Bc,Bn,rule,k", [(16, 16, orc.TOPK, 4), (32, 32, orc.TOPK, 8), (8, 24, orc.THRESHOLD, 0), (5, 3, orc.TOPK, 2),
                                          (1, 1, orc.THRESHOLD, 0)])
def test_commit_begin_step_equals_the_three_calls(shape, stream, Bc, Bn, rule, k):
    fused_case(shape, stream, Bc, Bn, rule, k)


def fused_case(shape, stream, Bc, Bn, rule, k, weight_seed=21):
    b = B_()
    tol = TOL[shape.dtype]
    st = torch.cuda.Stream() if stream else None
    oracle, handle, _ = make_pair(shape, weight_seed, max_seq=256, max_block=64, stream=st)
    emb, toks = I.make_prefix(shape, 12, 15, 6)
    oracle.prefill(I.as_numpy_storage(emb), toks.numpy(), want_logits=False)
    final = I.random_tokens(shape, Bc, 9)
    nxt_init = np.full(Bn, shape.mask_id, dtype=np.int64)
    if Bn >= 3:
        nxt_init[1] = int(I.random_tokens(shape, 1, 10)[0])          # one given token in the next block
    rule_code = b.RULE_THRESHOLD if rule == orc.THRESHOLD else b.RULE_TOPK
    dev = "cuda"
    g_next = torch.empty(shape.vocab, dtype=torch.float32, device=dev)
    g_logits = torch.empty(Bn, shape.vocab, dtype=torch.float32, device=dev)
    g_conf = torch.empty(Bn, dtype=torch.float32, device=dev)
    g_pred = torch.empty(Bn, dtype=torch.int32, device=dev)
    g_um = torch.empty(Bn, dtype=torch.uint8, device=dev)
    g_tok = torch.empty(Bn, dtype=torch.int32, device=dev)
    ctx = torch.cuda.stream(st) if st is not None else torch.cuda.stream(torch.cuda.current_stream())
    with ctx:
        handle.prefill(*upload_prefix(emb, toks))
        L0 = oracle.cache_len
        # a finished block on both sides
        oracle.block_begin(Bc, final.numpy())
        handle.block_begin(Bc, final.cuda())
        ref_next = oracle.commit_block()
        oracle.block_begin(Bn, nxt_init)
        rec = oracle.block_step(rule, 0.9, k)
        info = handle.commit_begin_step(Bn, rule_code, 0.9, k, next_logits=g_next,
                                        next_init_tokens=torch.from_numpy(nxt_init.astype(np.int32)).cuda(),
                                        logits=g_logits, conf=g_conf, pred=g_pred, unmask=g_um, block_tokens=g_tok)
        assert handle.cache_len() == oracle.cache_len == L0 + Bc and info.step_index == 1
        assert np.abs(g_next.double().cpu().numpy() - ref_next).max() <= tol["logits"]
        stats = {}
        compare_step(rec, g_logits, g_conf, g_pred, g_um, g_tok, info, shape, rule, 0.9, k, tol, stats)
        # the committed rows are the causal pass's
        for l in (0, shape.n_layers - 1):
            for which, ref in ((0, oracle.K[l]), (1, oracle.V[l])):
                got = handle.cache_read(l, which, L0, Bc).double().cpu().numpy()
                assert np.abs(got - ref[L0:L0 + Bc]).max() <= max(tol["logits"], 2e-2 * np.abs(ref[L0:]).max())
        # and the block state carries on: one more ordinary step from the oracle's state, if anything is left
        if oracle.masked.any():
            handle.block_set_tokens(torch.from_numpy(oracle.block_tokens.astype(np.int32)).cuda())
            rec2 = oracle.block_step(rule, 0.9, k)
            g2 = [torch.empty_like(t) for t in (g_logits, g_conf, g_pred, g_um, g_tok)]
            info2 = handle.block_step(rule_code, 0.9, k, logits=g2[0], conf=g2[1], pred=g2[2], unmask=g2[3], block_tokens=g2[4])
            compare_step(rec2, *g2, info2, shape, rule, 0.9, k, tol, stats)
    handle.close()


@pytest.mark.parametrize("rule,tau,k", [(orc.TOPK, 0.0, 4), (orc.THRESHOLD, 0.6, 0)])
def test_commit_decode_chain_matches_block_by_block_decoding_on_a_peaked_model(rule, tau, k):
    # three blocks: [steps, commit] x 3 against [commit fused into the next block's first step, remaining steps] x 3 (top-k:
    # fdvlm_commit_decode_block_topk; threshold: fdvlm_commit_decode_block, loop on the device).  The two ways run the same
    # arithmetic on other tile shapes, so tokens are compared only while the separate path's decisions are not near-ties.
    b = B_()
    shape, Bsz = SMALL_BF16, 16
    rule_code = b.RULE_TOPK if rule == orc.TOPK else b.RULE_THRESHOLD
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    _, ha, w = make_pair(shape, 33, max_seq=256, max_block=64, stream=sa, final_gain=16.0)
    hb = b.Handle(shape, b.weights_to_device(w), max_seq=256, max_block=64, stream=sb)
    emb, toks = I.make_prefix(shape, 10, 20, 5)
    blocks_a, blocks_b, steps_a, steps_b, clear = [], [], [], [], []
    with torch.cuda.stream(sa):
        ha.prefill(*upload_prefix(emb, toks))
        for _ in range(3):
            ha.block_begin(Bsz)
            ok, n = True, 0
            conf = torch.empty(Bsz, dtype=torch.float32, device="cuda")
            tok = torch.empty(Bsz, dtype=torch.int32, device="cuda")
            masked = np.ones(Bsz, dtype=bool)
            while masked.any():
                um = torch.empty(Bsz, dtype=torch.uint8, device="cuda")
                ha.block_step(rule_code, tau, k, conf=conf, unmask=um, block_tokens=tok)
                n += 1
                c = np.sort(conf.cpu().numpy()[masked])[::-1]
                if rule == orc.TOPK:
                    near = len(c) > k and c[k - 1] - c[k] <= 1e-5
                else:
                    near = np.any(np.abs(c - tau) <= 1e-5) or (c[0] <= tau and len(c) > 1 and c[0] - c[1] <= 1e-5)
                if near:
                    print("near-tie at step", n, "sorted confidences", c[:6])
                ok = ok and not near                                # (the two ways differ by ~1e-6 in confidence)
                masked &= ~um.cpu().numpy().astype(bool)
            blocks_a.append(tok.cpu().numpy().copy())
            steps_a.append(n)
            clear.append(ok)
            ha.commit_block()
    with torch.cuda.stream(sb):
        hb.prefill(*upload_prefix(emb, toks))
        L0 = hb.cache_len()
        for i in range(3):
            tok = torch.empty(Bsz, dtype=torch.int32, device="cuda")
            if rule == orc.TOPK:
                info = hb.commit_decode_block_topk(Bsz, k, block_tokens=tok)
            else:
                info = hb.commit_decode_block(Bsz, rule_code, tau, k, block_tokens=tok)
            assert info.n_remaining == 0 and 1 <= info.step_index <= Bsz
            assert hb.cache_len() == L0 + i * Bsz                 # the previous block went in with this call
            blocks_b.append(tok.cpu().numpy().copy())
            steps_b.append(info.step_index)
        hb.commit_block()
        assert hb.cache_len() == L0 + 3 * Bsz == ha.cache_len()
    assert clear[0]
    for a_, b_, na, nb, ok in zip(blocks_a, blocks_b, steps_a, steps_b, clear):
        if not ok:
            break                                                   # later blocks start from a different context
        assert np.array_equal(a_, b_) and na == nb
    ha.close()
    hb.close()


def test_fused_commit_state_and_capacity_errors():
    b = B_()
    _, handle, _ = make_pair(I.TINY, 1, max_seq=256, max_block=64)
    with pytest.raises(b.FdvlmError):
        handle.commit_begin_step(8, b.RULE_TOPK, 0.9, 4)             # nothing open
    handle.block_begin(8)
    with pytest.raises(b.FdvlmError):
        handle.commit_begin_step(8, b.RULE_TOPK, 0.9, 4)             # masked positions remain
    handle.block_step(b.RULE_THRESHOLD, -1.0, 0)                     # reveal everything
    with pytest.raises(b.FdvlmError) as e:
        handle.commit_begin_step(60, b.RULE_TOPK, 0.9, 4)            # 68 rows
    assert e.value.code == b.ERR_CAPACITY
    info = handle.commit_begin_step(8, b.RULE_TOPK, 0.9, 4)
    assert info.n_unmasked == 4 and info.n_remaining == 4 and handle.cache_len() == 8
    handle.close()
