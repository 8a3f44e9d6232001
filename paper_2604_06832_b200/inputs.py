"""Seeded synthetic inputs shared by the CUDA path's tests/bench and by the CPU oracle's tests.

This module holds NO arithmetic of the decoding method: it only draws random
numbers, casts them to the storage type of a configuration (fp32, bf16, or
FP8-E4M3 bytes plus per-output-channel fp32 scales) and describes the five
benchmark workloads.  Both sides receive the *same bytes*; each side decodes
bf16 / e4m3 bytes with code of its own.

Weight recipe (all workloads): every matrix ~ N(0, 0.02) drawn in fp32 from a
`torch.Generator` on the CPU, then cast; RMSNorm gains are 1.0 (optionally a
constant `final_gain` on the last norm, which only scales the logits and is used
by the "peaked" test variants so that confidences spread over (0, 1)).
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Dict, List, Optional

import torch

F32, BF16, FP8 = "f32", "bf16", "fp8"
W8A8 = "w8a8"      # weights stored as for FP8; the CUDA path also quantises the layer projections' input rows
E4M3_MAX = 448.0


@dataclass(frozen=True)
class ModelShape:
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    intermediate: int
    vocab: int
    mask_id: int
    rms_eps: float = 1e-6
    rope_theta: float = 1e6
    tie_embeddings: bool = True
    dtype: str = BF16          # storage type of the linear weights

    def with_(self, **kw) -> "ModelShape":
        return dataclasses.replace(self, **kw)

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def linear_elements(self) -> int:
        """Elements of every linear weight read once per forward (LM head included)."""
        per_layer = (self.hidden * (self.q_dim + 2 * self.kv_dim) + self.q_dim * self.hidden
                     + 3 * self.hidden * self.intermediate)
        return self.n_layers * per_layer + self.vocab * self.hidden

    def weight_bytes(self) -> int:
        esz = {F32: 4, BF16: 2, FP8: 1, W8A8: 1}[self.dtype]
        return self.linear_elements() * esz

    def kv_bytes_per_token(self) -> int:
        esz = 4 if self.dtype == F32 else 2
        return self.n_layers * 2 * self.kv_dim * esz


TINY = ModelShape(n_layers=2, hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, intermediate=688,
                  vocab=2048, mask_id=2047, tie_embeddings=True, dtype=F32)
QWEN3B = ModelShape(n_layers=36, hidden=2048, n_q_heads=16, n_kv_heads=2, head_dim=128,
                    intermediate=11008, vocab=151936, mask_id=151935, tie_embeddings=True, dtype=BF16)
QWEN7B_FP8 = ModelShape(n_layers=28, hidden=3584, n_q_heads=28, n_kv_heads=4, head_dim=128,
                        intermediate=18944, vocab=152064, mask_id=152063, tie_embeddings=False, dtype=FP8)


@dataclass(frozen=True)
class Workload:
    """One of the five benchmark configurations (index = position in the list, 1-based)."""
    name: str
    shape: ModelShape
    weight_seed: int
    prefix_seed: int
    n_embeds: int
    n_tokens: int
    new_tokens: int
    block_sizes: tuple
    rule: str                 # "threshold" | "topk"
    threshold: float = 0.9
    k: int = 8


WORKLOADS: Dict[str, Workload] = {
    "cfg1_tiny_f32": Workload("cfg1_tiny_f32", TINY, 0, 10, 48, 16, 8, (8,), "threshold"),
    "cfg2_3b_bf16_p1024_b32_top8": Workload("cfg2_3b_bf16_p1024_b32_top8", QWEN3B, 1, 12, 768, 256, 256, (32,), "topk"),
    "cfg3_3b_bf16_p2048_sweep": Workload("cfg3_3b_bf16_p2048_sweep", QWEN3B, 1, 13, 1536, 512, 256, (4, 8, 16, 32, 64), "threshold"),
    "cfg4_3b_bf16_p8192_b32_top8": Workload("cfg4_3b_bf16_p8192_b32_top8", QWEN3B, 1, 14, 7168, 1024, 512, (32,), "topk"),
    "cfg5_7b_fp8_p1024_b32": Workload("cfg5_7b_fp8_p1024_b32", QWEN7B_FP8, 5, 15, 768, 256, 256, (32,), "threshold"),
    # the 7B shape with the layer projections' inputs quantised per token as well (Sec. 3.4 "System integration")
    "w8a8_7b_p1024_b32": Workload("w8a8_7b_p1024_b32", QWEN7B_FP8.with_(dtype=W8A8), 5, 15, 768, 256, 256, (32,), "threshold"),
    # Profiler-sized cuts of the 3B / 7B shapes: same per-layer matrices, 4 layers and a 32768-row LM head, short
    # prefix.  About 0.75 GB (bf16) of weights per forward -- larger than L2, small enough for a counter capture.
    "prof_3b_bf16_4layers": Workload("prof_3b_bf16_4layers", QWEN3B.with_(n_layers=4, vocab=32768, mask_id=32767), 1, 16,
                                     96, 32, 64, (32,), "topk"),
    "prof_3b_bf16_4layers_p8192": Workload("prof_3b_bf16_4layers_p8192", QWEN3B.with_(n_layers=4, vocab=32768, mask_id=32767), 1, 18,
                                           7168, 1024, 64, (32,), "topk"),
    "prof_7b_fp8_4layers": Workload("prof_7b_fp8_4layers", QWEN7B_FP8.with_(n_layers=4, vocab=32768, mask_id=32767), 5, 17,
                                    96, 32, 64, (32,), "topk"),
    "prof_7b_w8a8_4layers": Workload("prof_7b_w8a8_4layers", QWEN7B_FP8.with_(n_layers=4, vocab=32768, mask_id=32767, dtype=W8A8), 5, 17,
                                     96, 32, 64, (32,), "topk"),
}


def _storage_dtype(dtype: str) -> torch.dtype:
    return torch.float32 if dtype == F32 else torch.bfloat16


def _normal(gen: torch.Generator, rows: int, cols: int, std: float = 0.02) -> torch.Tensor:
    return torch.empty(rows, cols, dtype=torch.float32, device=gen.device).normal_(0.0, std, generator=gen)


def quantize_e4m3_rows(w: torch.Tensor):
    """Per-output-channel FP8 storage of a [out, in] fp32 matrix.

    scale[n] = max_k |w[n,k]| / 448 (1.0 for an all-zero row); byte = e4m3fn(w / scale),
    round-to-nearest-even via torch's cast, saturating at +-448.  Returns (uint8 bytes, fp32 scales).
    """
    amax = w.abs().amax(dim=1)
    scale = torch.where(amax > 0, amax / E4M3_MAX, torch.ones_like(amax)).to(torch.float32)
    q = (w / scale[:, None]).clamp_(-E4M3_MAX, E4M3_MAX).to(torch.float8_e4m3fn)
    return q.view(torch.uint8), scale


def _store_linear(w: torch.Tensor, dtype: str):
    if dtype in (FP8, W8A8):
        return quantize_e4m3_rows(w)
    return w.to(_storage_dtype(dtype)), None


_LINEAR_NAMES = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")
_SCALE_NAMES = {"wq": "s_q", "wk": "s_k", "wv": "s_v", "wo": "s_o", "w_gate": "s_gate",
                "w_up": "s_up", "w_down": "s_down"}


def linear_dims(shape: ModelShape) -> Dict[str, tuple]:
    H, I = shape.hidden, shape.intermediate
    return {"wq": (shape.q_dim, H), "wk": (shape.kv_dim, H), "wv": (shape.kv_dim, H),
            "wo": (H, shape.q_dim), "w_gate": (I, H), "w_up": (I, H), "w_down": (H, I)}


def make_weights(shape: ModelShape, seed: int, *, qkv_bias: bool = False, final_gain: float = 1.0,
                 std: float = 0.02, device: str = "cpu", gain_spread: float = 0.0) -> dict:
    """All model weights as CPU tensors in storage dtype.

    Layout of the returned dict: 'embed' [vocab, hidden] (fp32 for an fp32 model, else bf16; never
    fp8), 'lm_head' / 's_lm_head' (None when tied), 'g_final' fp32 [hidden], 'layers': list of
    dicts with wq, wk, wv, wo, w_gate, w_up, w_down ([out, in] row-major), s_* fp32 [out] scales
    (fp8 only), optional fp32 biases bq, bk, bv, and fp32 gains g_attn, g_mlp.
    The draw order is fixed: embed, (lm_head), then per layer q, k, v, o, gate, up, down, (biases).
    `device` selects where the generator runs (the CPU stream is the one the parity tests use; a CUDA
    generator gives a different, equally seeded stream and is used by the bench for speed).
    `gain_spread` > 0 replaces the all-ones norm gains by 1 + gain_spread * U(-1, 1), drawn after everything else (so
    the other tensors do not change with it).
    """
    gen = torch.Generator(device=device).manual_seed(seed)
    H = shape.hidden
    out = {"shape": shape}
    out["embed"] = _normal(gen, shape.vocab, H, std).to(_storage_dtype(shape.dtype))
    if shape.tie_embeddings:
        out["lm_head"], out["s_lm_head"] = None, None
    else:
        out["lm_head"], out["s_lm_head"] = _store_linear(_normal(gen, shape.vocab, H, std), shape.dtype)
    out["g_final"] = torch.full((H,), float(final_gain), dtype=torch.float32, device=device)
    dims = linear_dims(shape)
    layers: List[dict] = []
    for _ in range(shape.n_layers):
        lw = {}
        for name in _LINEAR_NAMES:
            r, c = dims[name]
            lw[name], sc = _store_linear(_normal(gen, r, c, std), shape.dtype)
            lw[_SCALE_NAMES[name]] = sc
        for bname, wname in (("bq", "wq"), ("bk", "wk"), ("bv", "wv")):
            lw[bname] = (_normal(gen, 1, dims[wname][0], std).reshape(-1) if qkv_bias else None)
        lw["g_attn"] = torch.ones(H, dtype=torch.float32, device=device)
        lw["g_mlp"] = torch.ones(H, dtype=torch.float32, device=device)
        layers.append(lw)
    out["layers"] = layers
    if gain_spread > 0.0:
        draw = lambda: 1.0 + gain_spread * (2.0 * torch.rand(H, generator=gen, dtype=torch.float32, device=device) - 1.0)
        for lw in layers:
            lw["g_attn"], lw["g_mlp"] = draw(), draw()
        out["g_final"] = out["g_final"] * draw()
    return out


def make_prefix(shape: ModelShape, n_embeds: int, n_tokens: int, seed: int):
    """Vision-embedding rows ~ N(0,1) in the embedding table's dtype, and text tokens uniform over
    [0, vocab) with the mask id excluded."""
    gen = torch.Generator(device="cpu").manual_seed(seed)
    emb = torch.empty(n_embeds, shape.hidden, dtype=torch.float32).normal_(0.0, 1.0, generator=gen)
    emb = emb.to(_storage_dtype(shape.dtype))
    ids = torch.randint(0, shape.vocab - 1, (n_tokens,), generator=gen, dtype=torch.int64)
    ids = ids + (ids >= shape.mask_id).to(torch.int64)      # skip mask_id wherever it sits
    return emb, ids.to(torch.int32)


def random_tokens(shape: ModelShape, n: int, seed: int) -> torch.Tensor:
    gen = torch.Generator(device="cpu").manual_seed(seed)
    ids = torch.randint(0, shape.vocab - 1, (n,), generator=gen, dtype=torch.int64)
    ids = ids + (ids >= shape.mask_id).to(torch.int64)
    return ids.to(torch.int32)


def as_numpy_storage(t: Optional[torch.Tensor]):
    """View a storage tensor as a numpy array of raw storage: fp32 -> float32, bf16 -> uint16 bit
    patterns, fp8 bytes (already uint8) -> uint8.  No value conversion happens here."""
    if t is None:
        return None
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).numpy().view("uint16")
    return t.contiguous().numpy()


def weights_to_numpy(weights: dict) -> dict:
    """The same weights as raw numpy storage arrays (see `as_numpy_storage`); structure unchanged."""
    out = {k: as_numpy_storage(v) if isinstance(v, torch.Tensor) else v
           for k, v in weights.items() if k != "layers"}
    out["layers"] = [{k: as_numpy_storage(v) for k, v in lw.items()} for lw in weights["layers"]]
    return out
