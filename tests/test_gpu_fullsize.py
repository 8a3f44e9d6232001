"""GPU parity at the benchmark's full layer sizes, in the launch configuration `bench.py` times (a user stream, i.e.
graph replay + programmatic dependent launch, real tile counts, the full 151936-row LM head), at the STATED tolerances
(bf16 weights: logits 3e-2, confidence 5e-3; fp8 weights: 8e-2 / 1e-2).

The oracle needs ~13 s per forward of the 36-layer 3B shape, so the full-depth cases keep the prefix short (one 32-row
prefill chunk) and check one denoise step and the commit; the cases that need a long prefix or several block sizes use
4-layer cuts of the same shape (full per-layer matrices and full LM head, so every tile count is the real one)."""
import numpy as np
import pytest
import torch

from oracle import fdvlm_oracle as orc
from paper_2604_06832_b200 import inputs as I

from helpers import TOL, make_pair, replay_decode, upload_prefix

pytestmark = [pytest.mark.gpu, pytest.mark.slow]

CUT_3B = I.QWEN3B.with_(n_layers=4)


def B():
    from paper_2604_06832_b200 import binding
    return binding


def _short_prefix_case(shape, weight_seed, prefix_seed, n_blocks, kv_dtype, tol=None):
    stream = torch.cuda.Stream()
    oracle, handle, _ = make_pair(shape, weight_seed, max_seq=32 + 32 * n_blocks + 64, max_block=32, stream=stream,
                                  kv_dtype=kv_dtype)
    emb, toks = I.make_prefix(shape, 16, 16, prefix_seed)
    ref_last = oracle.prefill(I.as_numpy_storage(emb), toks.numpy())
    last = torch.empty(shape.vocab, dtype=torch.float32, device="cuda")
    tol = tol or TOL[shape.dtype]
    with torch.cuda.stream(stream):
        handle.prefill(*upload_prefix(emb, toks), last)
        stream.synchronize()
        prefill_err = float(np.abs(last.double().cpu().numpy() - ref_last).max())
        assert prefill_err <= tol["logits"], prefill_err
        # top-32 of 32 reveals the whole block in one step: one denoise forward and one commit per block
        stats = replay_decode(oracle, handle, shape, 32, orc.TOPK, 0.9, 32, n_blocks=n_blocks, tol=tol)
    assert stats["steps"] == n_blocks and handle.cache_len() == 32 + 32 * n_blocks
    handle.close()
    stats["prefill_err"] = prefill_err
    return stats


def test_full_36_layer_3b_shape_meets_the_stated_bf16_tolerance():
    wl = I.WORKLOADS["cfg2_3b_bf16_p1024_b32_top8"]
    stats = _short_prefix_case(wl.shape, wl.weight_seed, wl.prefix_seed, 1, B().KV_F16)
    print("3B x 36 layers, f16 cache: logit err", stats["logit_err"], "conf err", stats["conf_err"], "commit", stats["commit_err"])


def test_full_28_layer_7b_fp8_shape_meets_the_stated_fp8_tolerance():
    wl = I.WORKLOADS["cfg5_7b_fp8_p1024_b32"]
    stats = _short_prefix_case(wl.shape, wl.weight_seed, wl.prefix_seed, 1, B().KV_F16)
    print("7B fp8 x 28 layers, f16 cache: logit err", stats["logit_err"], "conf err", stats["conf_err"], "commit", stats["commit_err"])


@pytest.mark.xfail(strict=False, reason="bf16 K/V rounding alone exceeds the stated logit bound at this depth; "
                                        "the f16-cache handle (test above) differs in this one setting and meets it")
@pytest.mark.parametrize("wl_name", ["cfg2_3b_bf16_p1024_b32_top8", "cfg5_7b_fp8_p1024_b32"])
def test_full_depth_with_a_bf16_cache_records_its_error(wl_name):
    """The one-variable experiment behind the kv_dtype setting: same weights, same inputs, same kernels, only the element
    type of q / K / V / attention probabilities changed to bf16.  Asserts the stated bound (expected to fail: the measured
    error is the record)."""
    wl = I.WORKLOADS[wl_name]
    stats = _short_prefix_case(wl.shape, wl.weight_seed, wl.prefix_seed, 1, B().KV_BF16, tol=dict(logits=10.0, conf=1.0))
    print(wl_name, "bf16 cache: logit err", stats["logit_err"], "conf err", stats["conf_err"], "commit", stats["commit_err"])
    assert max(stats["logit_err"], stats["commit_err"], stats["prefill_err"]) <= TOL[wl.shape.dtype]["logits"]


def test_fp8_4_layer_cut_two_blocks():
    wl = I.WORKLOADS["prof_7b_fp8_4layers"]
    _short_prefix_case(wl.shape, wl.weight_seed, wl.prefix_seed, 2, B().KV_BF16)


@pytest.mark.parametrize("block", [4, 8, 16, 64])
def test_block_size_sweep_on_the_4_layer_cut_at_prefix_2048(block):
    """Every activation-tile width of the GEMM (16 / 32 / 48 / 64 rows hold blocks of 4-16 / 32 / - / 64) at the real tile
    counts of the 3B matrices, behind the 2048-position prefix of the block-size sweep."""
    wl = I.WORKLOADS["cfg3_3b_bf16_p2048_sweep"]
    stream = torch.cuda.Stream()
    oracle, handle, _ = make_pair(CUT_3B, wl.weight_seed, max_seq=2048 + 2 * block, max_block=64, stream=stream)
    emb, toks = I.make_prefix(CUT_3B, wl.n_embeds, wl.n_tokens, wl.prefix_seed)
    oracle.prefill(I.as_numpy_storage(emb), toks.numpy(), want_logits=False)
    with torch.cuda.stream(stream):
        handle.prefill(*upload_prefix(emb, toks))
        stats = replay_decode(oracle, handle, CUT_3B, block, orc.TOPK, 0.9, max(block // 2, 1), n_blocks=2)
    assert stats["steps"] == 4 and handle.cache_len() == 2048 + 2 * block
    handle.close()


def test_long_prefix_8192_end_to_end_on_the_4_layer_cut():
    """Prefill of 7168 embedding rows + 1024 tokens, a denoise step and the commit behind it; the committed cache rows
    are compared too."""
    wl = I.WORKLOADS["cfg4_3b_bf16_p8192_b32_top8"]
    stream = torch.cuda.Stream()
    oracle, handle, _ = make_pair(CUT_3B, wl.weight_seed, max_seq=8192 + 64, max_block=32, stream=stream)
    emb, toks = I.make_prefix(CUT_3B, wl.n_embeds, wl.n_tokens, wl.prefix_seed)
    ref_last = oracle.prefill(I.as_numpy_storage(emb), toks.numpy())
    last = torch.empty(CUT_3B.vocab, dtype=torch.float32, device="cuda")
    with torch.cuda.stream(stream):
        handle.prefill(*upload_prefix(emb, toks), last)
        stream.synchronize()
        assert np.abs(last.double().cpu().numpy() - ref_last).max() <= TOL[I.BF16]["logits"]
        for layer in (0, 3):
            for which, ref in ((0, oracle.K[layer]), (1, oracle.V[layer])):
                for pos0 in (0, 5000, 8192 - 64):
                    got = handle.cache_read(layer, which, pos0, 64)
                    stream.synchronize()
                    err = np.abs(got.double().cpu().numpy() - ref[pos0:pos0 + 64])
                    assert (err <= 2e-3 * np.maximum(np.abs(ref[pos0:pos0 + 64]), 1.0)).all()      # f16 storage: 2^-11 relative
        stats = replay_decode(oracle, handle, CUT_3B, 32, orc.TOPK, 0.9, 8, n_blocks=1)
        got = handle.cache_read(3, 0, 8192, 32)
        stream.synchronize()
    assert stats["steps"] == 4 and handle.cache_len() == 8192 + 32
    ref = oracle.K[3][8192:8192 + 32]
    assert (np.abs(got.double().cpu().numpy() - ref) <= 2e-3 * np.maximum(np.abs(ref), 1.0)).all()
    handle.close()


def test_prefix_1024_on_the_4_layer_cut_with_the_benchmark_schedule():
    wl = I.WORKLOADS["cfg2_3b_bf16_p1024_b32_top8"]
    stream = torch.cuda.Stream()
    oracle, handle, _ = make_pair(CUT_3B, wl.weight_seed, max_seq=1024 + 64, max_block=32, stream=stream)
    emb, toks = I.make_prefix(CUT_3B, wl.n_embeds, wl.n_tokens, wl.prefix_seed)
    oracle.prefill(I.as_numpy_storage(emb), toks.numpy(), want_logits=False)
    with torch.cuda.stream(stream):
        handle.prefill(*upload_prefix(emb, toks))
        stats = replay_decode(oracle, handle, CUT_3B, 32, orc.TOPK, 0.9, 8, n_blocks=2)
    assert stats["steps"] == 8 and handle.cache_len() == 1024 + 64
    handle.close()


def test_peaked_3b_width_model_discrete_parity_is_not_vacuous():
    """Same widths, final gain raised so that confidences spread over (0, 1): rows with a clear top-2 margin exist and
    whole steps have clear selection decisions, so the token / unmask-set comparison really runs at this width."""
    gain = 12.0
    stream = torch.cuda.Stream()
    oracle, handle, _ = make_pair(CUT_3B, 1, max_seq=160, max_block=32, stream=stream, final_gain=gain)
    emb, toks = I.make_prefix(CUT_3B, 40, 24, 12)
    oracle.prefill(I.as_numpy_storage(emb), toks.numpy(), want_logits=False)
    # logits (and their errors) scale with the gain; a probability near 1/2 moves by a quarter of the logit error
    tol = dict(logits=TOL[I.BF16]["logits"] * gain, conf=TOL[I.BF16]["logits"] * gain / 4, gap=2 * TOL[I.BF16]["logits"] * gain)
    with torch.cuda.stream(stream):
        handle.prefill(*upload_prefix(emb, toks))
        stats = replay_decode(oracle, handle, CUT_3B, 32, orc.THRESHOLD, 0.9, 0, n_blocks=2, tol=tol)
    print("peaked 3B-width cut:", stats)
    assert stats.get("rows_sure", 0) > 0 and stats.get("steps_clear", 0) > 0
    handle.close()


def test_attention_at_the_long_prefix_length():
    """The split-KV kernel at the 8192-position prefix of the long-context configuration (16 query / 2 KV heads)."""
    n, L, hq, hkv, d = 32, 8192, 16, 2, 128
    g = torch.Generator().manual_seed(4)
    for td, bound in ((torch.bfloat16, 2e-2), (torch.float16, 3e-3)):
        q = torch.randn(n, hq, d, generator=g).to(td)
        kc = torch.randn(hkv, L + n, d, generator=g).to(td)
        vc = torch.randn(hkv, L + n, d, generator=g).to(td)
        f = lambda t: t.double().numpy()
        for causal in (0, 1):
            allowed = np.ones((n, L + n), dtype=bool)
            if causal:
                allowed[:, L:] = np.tril(np.ones((n, n), dtype=bool))
            ref = orc.attend(f(q), f(kc).transpose(1, 0, 2), f(vc).transpose(1, 0, 2), allowed).reshape(n, hq * d)
            out = B().op_attention(q.cuda(), kc.cuda(), vc.cuda(), L, bool(causal), dtype=B().DT_BF16)
            torch.cuda.synchronize()
            assert np.abs(out.double().cpu().numpy() - ref).max() <= bound


# ---- the fused commit, Alg. 2's masked forward and the W8A8 projection at the real layer widths -------------------
@pytest.mark.parametrize("shape", [CUT_3B, I.QWEN7B_FP8.with_(n_layers=4)], ids=["3b-bf16-cut", "7b-fp8-cut"])
def test_fused_commit_at_full_width(shape):
    from test_gpu_fused_commit import fused_case
    fused_case(shape, True, 32, 32, orc.TOPK, 8)          # the 64-row forward the bench's top-k workloads run


def test_fused_commit_at_full_depth_is_the_forward_the_bench_times():
    # cfg2's model, all 36 layers: the 64-row forward (commit of one block + first top-8 step of the next) at the stated bounds
    from test_gpu_fused_commit import fused_case
    wl = I.WORKLOADS["cfg2_3b_bf16_p1024_b32_top8"]
    fused_case(wl.shape, True, 32, 32, orc.TOPK, 8, weight_seed=wl.weight_seed)


def test_quadratic_decoding_at_full_width():
    from test_gpu_quad import run_iterations
    stats = run_iterations(CUT_3B, 7, False, n_iter=1, stream=True)      # 56 rows, the largest block one forward takes
    print("quadratic, 3B-width cut:", stats)


@pytest.mark.parametrize("n,k", [(3584 + 2 * 512, 3584), (3584, 18944), (2 * 18944, 3584)], ids=["qkv", "down", "gate-up"])
def test_w8a8_projection_at_the_7b_shapes(n, k):
    from test_gpu_w8a8 import test_op_linear_w8a8_quantises_like_the_oracle as case
    case(32, n, k)

