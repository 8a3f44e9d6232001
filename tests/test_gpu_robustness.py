"""GPU tests of what surrounds the arithmetic: the give-up path of the kernels' bounded waits (driven by a host-set flag,
never by a real hang), out-of-range token ids, the on-device decode loop against the step-by-step path, the in-chain
timing records, and handles on a second stream in one process."""
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


@pytest.mark.parametrize("shape", [SMALL_BF16, SMALL_FP8])
@pytest.mark.parametrize("on_stream", [False, True])
def test_give_up_path_of_the_bounded_waits(shape, on_stream):
    """With the poison flag set every role of every GEMM leaves by the branch a timed-out wait takes (nothing issued,
    tensor memory freed): the call reports FDVLM_ERR_TIMEOUT, the committed cache is untouched, and once the flag is
    cleared the same handle matches the oracle again."""
    b = B()
    stream = torch.cuda.Stream() if on_stream else None
    oracle, handle, _ = make_pair(shape, 31, max_seq=200, stream=stream)
    emb, toks = I.make_prefix(shape, 20, 13, 8)
    oracle.prefill(I.as_numpy_storage(emb), toks.numpy(), want_logits=False)
    ctx = torch.cuda.stream(stream) if on_stream else torch.cuda.stream(torch.cuda.current_stream())
    with ctx:
        handle.prefill(*upload_prefix(emb, toks))
        handle.synchronize()
        before = [handle.cache_read(l, w, 0, 33).clone() for l in range(shape.n_layers) for w in (0, 1)]
        handle.debug_poison(True)
        handle.block_begin(16)
        with pytest.raises(b.FdvlmError) as e:
            handle.block_step(b.RULE_TOPK, 0.0, 4)
        assert e.value.code == b.ERR_TIMEOUT and "gave up" in str(e.value)
        after = [handle.cache_read(l, w, 0, 33) for l in range(shape.n_layers) for w in (0, 1)]
        torch.cuda.synchronize()
        assert all(torch.equal(x, y) for x, y in zip(before, after))
        # a poisoned asynchronous call reports through fdvlm_synchronize
        handle.reset()
        handle.prefill(*upload_prefix(emb, toks))
        with pytest.raises(b.FdvlmError) as e:
            handle.synchronize()
        assert e.value.code == b.ERR_TIMEOUT
        handle.debug_poison(False)
        handle.reset()
        handle.prefill(*upload_prefix(emb, toks))
        handle.synchronize()
        stats = replay_decode(oracle, handle, shape, 16, orc.TOPK, 0.9, 4, n_blocks=2)
    assert stats["steps"] == 8
    handle.close()


def test_poisoned_operator_call_reports_through_its_status_query():
    b = B()
    m, n, k = 32, 1024, 512
    x = torch.randn(m, k).to(torch.bfloat16).cuda()
    w = (torch.randn(n, k) * 0.05).to(torch.bfloat16).cuda()
    y = torch.zeros(m, n, dtype=torch.float32, device="cuda")
    ws = torch.zeros(b.lib().fdvlm_op_linear_workspace_bytes(m, n, k, b.DT_BF16), dtype=torch.uint8, device="cuda")
    assert b.lib().fdvlm_op_linear(x.data_ptr(), w.data_ptr(), None, None, y.data_ptr(), m, n, k, b.DT_BF16, ws.data_ptr(), None) == 0
    assert b.lib().fdvlm_op_linear_status(ws.data_ptr(), None) == 0
    ref = x.float() @ w.float().T
    assert float((y - ref).abs().max()) <= 2e-4 * float(ref.abs().max())


@pytest.mark.parametrize("shape", [I.TINY, SMALL_BF16])
def test_token_ids_out_of_range_are_reported_not_dereferenced(shape):
    b = B()
    _, handle, _ = make_pair(shape, 3, max_seq=64, max_block=8)
    bad = torch.tensor([1, 2, shape.vocab + 5, 3], dtype=torch.int32, device="cuda")
    handle.prefill(None, bad)
    with pytest.raises(b.FdvlmError) as e:
        handle.synchronize()
    assert e.value.code == b.ERR_INVALID_ARG and "token" in str(e.value)
    handle.reset()
    init = torch.tensor([5, -7, shape.mask_id, shape.mask_id], dtype=torch.int32, device="cuda")
    handle.block_begin(4, init)
    with pytest.raises(b.FdvlmError) as e:
        handle.block_step(b.RULE_TOPK, 0.0, 2)
    assert e.value.code == b.ERR_INVALID_ARG
    # the report is consumed: a clean request on the same handle works
    handle.reset()
    handle.prefill(None, I.random_tokens(shape, 6, 1).cuda())
    handle.synchronize()
    handle.close()


@pytest.mark.parametrize("shape,gain,rule,tau,k,shift", [
    (SMALL_BF16, 16.0, orc.THRESHOLD, 0.6, 0, 0), (SMALL_BF16, 1.0, orc.THRESHOLD, 0.9, 0, 0), (SMALL_BF16, 16.0, orc.TOPK, 0.0, 5, 0),
    (SMALL_FP8, 12.0, orc.THRESHOLD, 0.5, 0, 1), (SMALL_BF16, 1.0, orc.THRESHOLD, -1.0, 0, 0)])
def test_on_device_decode_loop_equals_the_step_by_step_path(shape, gain, rule, tau, k, shift):
    """fdvlm_decode_block runs the whole denoise loop of a block inside one graph launch (a conditional WHILE node);
    its block tokens and step count must be those of fdvlm_block_step called until no mask is left -- bit for bit, the
    kernels being the same -- and on a peaked model the threshold rule must really take fewer steps than positions."""
    b = B()
    B_ = 16
    stream = torch.cuda.Stream()
    _, handle, w = make_pair(shape, 17, max_seq=128, stream=stream, final_gain=gain)
    emb, toks = I.make_prefix(shape, 24, 9, 2)
    code = b.RULE_THRESHOLD if rule == orc.THRESHOLD else b.RULE_TOPK
    init = None
    if shift:
        init = torch.full((B_,), shape.mask_id, dtype=torch.int32)
        init[0] = 11
        init = init.cuda()
    with torch.cuda.stream(stream):
        handle.prefill(*upload_prefix(emb, toks))
        ref_tokens = torch.empty(B_, dtype=torch.int32, device="cuda")
        handle.block_begin(B_, init)
        steps = 0
        while True:
            info = handle.block_step(code, tau, k, block_tokens=ref_tokens, pred_shift=shift)
            steps += 1
            if info.n_remaining == 0:
                break
        ref_tokens = ref_tokens.clone()
        handle.commit_block()
        handle.truncate(33)                              # same cache for the second run
        got = torch.empty(B_, dtype=torch.int32, device="cuda")
        info = handle.decode_block(B_, code, tau, k, init_tokens=init, pred_shift=shift, block_tokens=got)
        stream.synchronize()
        assert info.n_remaining == 0 and info.step_index == steps
        assert torch.equal(got, ref_tokens)
        nxt = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
        handle.commit_block(nxt)
        # a second block through the kept loop graph, at a longer cache
        info2 = handle.decode_block(B_, code, tau, k, init_tokens=init, pred_shift=shift, block_tokens=got)
        assert info2.n_remaining == 0 and 1 <= info2.step_index <= B_
        handle.commit_block()
    assert handle.cache_len() == 33 + 2 * B_
    if rule == orc.THRESHOLD and tau < 0:
        assert steps == 1
    if rule == orc.TOPK:
        assert steps == -(-B_ // k)
    if gain > 1.0 and rule == orc.THRESHOLD:
        assert steps < B_ - shift, "peaked model: some step should reveal several positions"
    handle.close()


def test_decode_loop_needs_a_user_stream():
    b = B()
    _, handle, _ = make_pair(SMALL_BF16, 17, max_seq=64)
    with pytest.raises(b.FdvlmError) as e:
        handle.decode_block(8, b.RULE_THRESHOLD, 0.9)
    assert e.value.code == b.ERR_UNSUPPORTED
    handle.close()


def test_in_chain_timing_records_are_consistent():
    """Profile mode 2: every kernel of the replayed forward leaves (start, released, end) from the GPU's timer.  The
    records come in launch order, each kernel ends after it starts, a kernel is released only after its predecessor has
    ended, and the outputs are bit-identical to an unprofiled step."""
    b = B()
    shape = SMALL_BF16
    stream = torch.cuda.Stream()
    _, handle, _ = make_pair(shape, 5, max_seq=128, stream=stream)
    emb, toks = I.make_prefix(shape, 24, 8, 2)
    lg = [torch.empty(16, shape.vocab, dtype=torch.float32, device="cuda") for _ in range(2)]
    with torch.cuda.stream(stream):
        handle.prefill(*upload_prefix(emb, toks))
        handle.block_begin(16)
        handle.block_step(b.RULE_TOPK, 0.0, 16, logits=lg[0])
        handle.block_set_tokens(torch.full((16,), shape.mask_id, dtype=torch.int32, device="cuda"))
        handle.profile_enable(2)
        handle.block_step(b.RULE_TOPK, 0.0, 16, logits=lg[1])
        recs = handle.profile_read_chain()
        handle.profile_enable(0)
        stream.synchronize()
    assert torch.equal(lg[0], lg[1])
    kinds = [r["kind"] for r in recs]
    per_layer = ["gemm_qkv", "fin_qkv", "attention", "attn_merge", "gemm_o", "fin_resid", "gemm_gate_up", "gemm_down", "fin_resid"]
    assert kinds == ["rope_table"] + per_layer * shape.n_layers + ["gemm_lm_head", "stats_merge"]
    prev_end = None
    for r in recs:
        assert 0 <= r["start_us"] <= r["end_us"], r
        if r["released_us"] >= 0:
            assert r["start_us"] <= r["released_us"] <= r["end_us"], r
            if prev_end is not None:
                assert r["released_us"] >= prev_end - 0.5, (r, prev_end)     # half a microsecond for timer granularity
        prev_end = r["end_us"]
    assert recs[-1]["end_us"] < 5e4
    handle.close()


def test_two_handles_on_two_streams_in_one_process():
    shape = SMALL_BF16
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    o1, h1, _ = make_pair(shape, 41, max_seq=128, stream=s1)
    o2, h2, _ = make_pair(shape, 42, max_seq=128, stream=s2)
    emb, toks = I.make_prefix(shape, 10, 10, 3)
    for o in (o1, o2):
        o.prefill(I.as_numpy_storage(emb), toks.numpy(), want_logits=False)
    with torch.cuda.stream(s1):
        h1.prefill(*upload_prefix(emb, toks))
    with torch.cuda.stream(s2):
        h2.prefill(*upload_prefix(emb, toks))
    with torch.cuda.stream(s1):
        st1 = replay_decode(o1, h1, shape, 8, orc.TOPK, 0.9, 4)
    with torch.cuda.stream(s2):
        st2 = replay_decode(o2, h2, shape, 8, orc.TOPK, 0.9, 4)
    assert st1["steps"] == st2["steps"] == 2
    h1.close()
    h2.close()


def test_stream_read_yardstick_runs_and_rejects_bad_arguments():
    b = B()
    buf = torch.zeros(64 << 20, dtype=torch.uint8, device="cuda")
    sink = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.util_stream_read(buf, sink)
    torch.cuda.synchronize()
    assert int(sink.item()) == 0                                   # all-zero data never folds to the magic word
    with pytest.raises(b.FdvlmError):
        b.util_stream_read(buf[1:], sink)                          # not 16-byte aligned
    assert b.lib().fdvlm_util_stream_read(None, 1024, sink.data_ptr(), None) == b.ERR_INVALID_ARG
