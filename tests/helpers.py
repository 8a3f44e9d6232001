"""Shared helpers of the GPU parity tests: build the oracle and the CUDA handle from the same seeded
bytes and compare one decode, step by step, in replay mode (the CUDA path is handed the oracle's block
state before every step so a single low-margin token cannot cascade)."""
import numpy as np
import torch

from oracle import fdvlm_oracle as orc
from paper_2604_06832_b200 import inputs as I

TOL = {I.F32: dict(logits=1e-4, conf=1e-4), I.BF16: dict(logits=3e-2, conf=5e-3), I.FP8: dict(logits=8e-2, conf=1e-2)}
MARGIN = 1e-3


def make_pair(shape, seed, max_seq, max_block=64, stream=None, kv_dtype=None, **wkw):
    """`stream`: a torch.cuda.Stream for the handle (the library then replays captured CUDA graphs; on the default
    stream it launches kernel by kernel).  `kv_dtype`: binding.KV_F16 (default) or binding.KV_BF16."""
    from paper_2604_06832_b200 import binding as B
    w = I.make_weights(shape, seed, **wkw)
    oracle = orc.Oracle(shape, I.weights_to_numpy(w))
    handle = B.Handle(shape, B.weights_to_device(w), max_seq=max_seq, max_block=max_block, stream=stream,
                      kv_dtype=B.KV_F16 if kv_dtype is None else kv_dtype)
    return oracle, handle, w


def decisions_clear(rec, rule, threshold, k, tol_conf):
    """True when no selection decision of this step sits within the confidence tolerance."""
    conf, masked = rec["conf"], rec["masked_before"]
    idx = np.flatnonzero(masked)
    if idx.size == 0:
        return True
    c = np.sort(conf[idx])[::-1]
    if rule == orc.THRESHOLD:
        if np.any(np.abs(conf[idx] - threshold) <= tol_conf):
            return False
        if not np.any(conf[idx] > threshold):           # argmax fallback: top-1 vs top-2 gap
            return idx.size == 1 or (c[0] - c[1]) > 2 * tol_conf
        return True
    kk = min(k, idx.size)
    return kk == idx.size or (c[kk - 1] - c[kk]) > 2 * tol_conf


def compare_step(rec, g_logits, g_conf, g_pred, g_unmask, g_tokens, info, shape, rule, threshold, k, tol, stats):
    logits = g_logits.double().cpu().numpy()
    err = np.abs(logits - rec["logits"]).max()
    stats["logit_err"] = max(stats.get("logit_err", 0.0), float(err))
    assert err <= tol["logits"], f"logits max-abs err {err}"
    conf = g_conf.double().cpu().numpy()
    m = rec["masked_before"]
    cerr = np.abs(conf - rec["conf"])[m].max()
    stats["conf_err"] = max(stats.get("conf_err", 0.0), float(cerr))
    assert cerr <= tol["conf"], f"conf err {cerr}"
    pred = g_pred.cpu().numpy()
    sure = rec["margin"] > MARGIN
    if "gap" in tol:   # supplementary scaled-logit variants: also require a top-2 logit gap beyond the logit error bound
        l = rec["logits"].copy()
        l[:, shape.mask_id] = -np.inf
        top2 = np.sort(l, axis=1)[:, -2:]
        sure = sure & ((top2[:, 1] - top2[:, 0]) > tol["gap"])
    stats["rows_sure"] = stats.get("rows_sure", 0) + int(sure.sum())
    assert np.array_equal(pred[sure], rec["pred"][sure]), "token ids differ where the top-2 margin is clear"
    assert (pred != shape.mask_id).all()
    um = g_unmask.cpu().numpy().astype(bool)
    assert not (um & ~m).any() and um.sum() >= 1 and info.n_unmasked == um.sum()
    if decisions_clear(rec, rule, threshold, k, tol["conf"]):
        stats["steps_clear"] = stats.get("steps_clear", 0) + 1
        assert np.array_equal(um, rec["unmask"]), "unmask sets differ although every decision is clear"
        assert info.n_remaining == rec["n_remaining"]
        toks = g_tokens.cpu().numpy()
        ok = ~um | sure
        assert np.array_equal(toks[ok], rec["block_tokens"][ok])


def replay_decode(oracle, handle, shape, block_size, rule, threshold=0.9, k=8, n_blocks=1, tol=None, check_commit=True):
    """Decode n_blocks blocks on both sides in replay mode; returns error statistics."""
    from paper_2604_06832_b200 import binding as B
    tol = tol or TOL[shape.dtype]
    stats = {"steps": 0}
    dev = "cuda"
    Bsz = block_size
    g_logits = torch.empty(Bsz, shape.vocab, dtype=torch.float32, device=dev)
    g_conf = torch.empty(Bsz, dtype=torch.float32, device=dev)
    g_pred = torch.empty(Bsz, dtype=torch.int32, device=dev)
    g_unmask = torch.empty(Bsz, dtype=torch.uint8, device=dev)
    g_tokens = torch.empty(Bsz, dtype=torch.int32, device=dev)
    nxt = torch.empty(shape.vocab, dtype=torch.float32, device=dev)
    rule_code = B.RULE_THRESHOLD if rule == orc.THRESHOLD else B.RULE_TOPK
    for _ in range(n_blocks):
        oracle.block_begin(Bsz)
        handle.block_begin(Bsz)
        while oracle.masked.any():
            state = torch.from_numpy(oracle.block_tokens.astype(np.int32)).to(dev)
            handle.block_set_tokens(state)
            rec = oracle.block_step(rule, threshold, k)
            info = handle.block_step(rule_code, threshold, k, logits=g_logits, conf=g_conf, pred=g_pred,
                                     unmask=g_unmask, block_tokens=g_tokens)
            compare_step(rec, g_logits, g_conf, g_pred, g_unmask, g_tokens, info, shape, rule, threshold, k, tol, stats)
            stats["steps"] += 1
        final = torch.from_numpy(oracle.block_tokens.astype(np.int32)).to(dev)
        handle.block_set_tokens(final)
        ref_next = oracle.commit_block()
        handle.commit_block(nxt)
        assert handle.cache_len() == oracle.cache_len
        if check_commit:
            err = np.abs(nxt.double().cpu().numpy() - ref_next).max()
            stats["commit_err"] = max(stats.get("commit_err", 0.0), float(err))
            assert err <= tol["logits"], f"commit logits err {err}"
    return stats


def upload_prefix(emb, toks):
    return (emb.cuda() if emb is not None and len(emb) else None), (toks.cuda() if toks is not None and len(toks) else None)
