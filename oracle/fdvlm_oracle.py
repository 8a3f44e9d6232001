"""CPU oracle for the block-diffusion denoise step -- TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 numpy statement of what one request at batch size one computes:
causal prefill, the bidirectional-in-block denoise forward over the committed KV cache,
softmax-max confidence, threshold / top-k unmasking, and the causal commit of a finished
block.  It shares no code with the CUDA library and is never imported by it; only the
tests, the smoke check and the bench's CPU-baseline leg may use it.

Paper passages each function follows are named in its docstring (section / algorithm).
Where the paper is silent the reading taken is stated next to the code.

Pinned by tests that do not call back into this file's own formulas: B=1 == causal AR,
chunked prefill + commit == one dense causal pass, cached path == dense brute-force mask,
dependency probes, selection closed forms, softmax identities, GQA == MHA with repeated
K/V weights, RoPE shift invariance, RMSNorm / SwiGLU closed forms, hand-checkable
zero-layer logits, an independent torch restatement of attention, a hand-worked e4m3 matrix
with per-row scales, and the untied FP8 LM head recomputed row by row; planted errors (a rotation
sign, a scale on the wrong axis, an ignored head or head scale) must make those pins fail.
Parity unpinned: absolute logit values of the random-init models (the paper prints no
worked numerical example of a denoise step).
"""
from __future__ import annotations

import numpy as np

NEG_INF = -np.inf

THRESHOLD, TOPK = "threshold", "topk"
BIDIR, CAUSAL = "bidir", "causal"


# ----------------------------------------------------------------------------------------------
# storage decoding (bf16: upper half of an IEEE fp32; e4m3: OCP "e4m3fn": 1-4-3, bias 7, no inf,
# S.1111.111 = NaN, max 448)
# ----------------------------------------------------------------------------------------------
def decode_bf16(bits: np.ndarray) -> np.ndarray:
    assert bits.dtype == np.uint16
    with np.errstate(invalid="ignore"):
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def _e4m3_table() -> np.ndarray:
    t = np.zeros(256, dtype=np.float64)
    for b in range(256):
        s = -1.0 if (b >> 7) else 1.0
        e = (b >> 3) & 0xF
        m = b & 0x7
        if e == 0xF and m == 0x7:
            v = np.nan
        elif e == 0:
            v = (m / 8.0) * 2.0 ** (-6)
        else:
            v = (1.0 + m / 8.0) * 2.0 ** (e - 7)
        t[b] = s * v
    return t


_E4M3 = _e4m3_table()


def decode_e4m3(bits: np.ndarray) -> np.ndarray:
    assert bits.dtype == np.uint8
    return _E4M3[bits]


def round_e4m3(v: np.ndarray) -> np.ndarray:
    """Nearest OCP e4m3fn value of every element (ties to the even mantissa), saturating at +-448.

    The format has 3 mantissa bits, normal exponents 2^-6 .. 2^8 and subnormals in steps of 2^-9, so the spacing at
    |v| in [2^e, 2^(e+1)) is 2^(e-3) with e clamped to >= -6.  Input and the rounding decision are float32 (the type
    in which the quantised path forms the value it rounds); the result is returned exactly, as float64."""
    v = np.asarray(v, dtype=np.float32)
    a = np.abs(v)
    _, ex = np.frexp(a)                                  # a = m * 2^ex, m in [0.5, 1)
    e = np.clip(ex.astype(np.int32) - 1, -6, 8)
    quantum = np.ldexp(np.float32(1.0), e - 3).astype(np.float32)
    q = np.rint(a / quantum) * quantum                   # power-of-two scaling: exact; rint rounds half to even
    q = np.minimum(q, np.float32(448.0))
    return np.copysign(q, v).astype(np.float64)


def quantize_rows_e4m3(a: np.ndarray) -> np.ndarray:
    """Per-token (per-row) dynamic FP8 quantisation of an activation matrix, returned de-quantised.

    scale_r = max_k |a_rk| / 448 (1 for an all-zero row), code = e4m3(a / scale_r), value = code * scale_r: the
    activation half of the W8A8 setting of Sec. 3.4 "System integration" / Sec. 4.5 (the smoothing of SmoothQuant is a
    per-channel rescaling folded into the preceding norm gain and the weights offline, so nothing of it is left at run
    time).  The row maximum, the scale, the quotient and the rounding are taken in float32."""
    a32 = np.asarray(a, dtype=np.float32)
    amax = np.max(np.abs(a32), axis=-1, keepdims=True)
    scale = np.where(amax > 0, amax / np.float32(448.0), np.float32(1.0)).astype(np.float32)
    codes = round_e4m3(a32 / scale)
    return codes * scale.astype(np.float64)


def to_f64(a: np.ndarray) -> np.ndarray:
    """Exact value of a storage array: float32/float64 as is, uint16 = bf16 bits, uint8 = e4m3 bits."""
    if a.dtype == np.uint16:
        return decode_bf16(a)
    if a.dtype == np.uint8:
        return decode_e4m3(a)
    return a.astype(np.float64)


# ----------------------------------------------------------------------------------------------
# elementary operators (Qwen2.5-style pre-norm decoder, the backbone of Sec. 4.1 / App. A.2)
# ----------------------------------------------------------------------------------------------
def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """x * rsqrt(mean(x^2) + eps) * g, row-wise."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, rotate-half pairing (j, j + d/2), angle = pos * theta^(-2j/d).

    x: [n, heads, d]; pos: [n] integer positions in the committed sequence (the paper is silent on
    the form; this is the 1-D rotary form of the Qwen2.5 decoder family)."""
    n, _, d = x.shape
    half = d // 2
    j = np.arange(half, dtype=np.float64)
    inv_freq = theta ** (-2.0 * j / d)
    ang = pos.astype(np.float64)[:, None] * inv_freq[None, :]          # [n, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def attend(q: np.ndarray, k: np.ndarray, v: np.ndarray, allowed: np.ndarray) -> np.ndarray:
    """softmax(q k^T / sqrt(d)) v over the allowed keys, grouped-query heads.

    q: [n, Hq, d]; k, v: [T, Hkv, d]; allowed: bool [n, T] (M_N2N / M_N2C / M_C2C of Sec. 3.3 are
    all expressed through it).  Query head h reads KV head h // (Hq / Hkv)."""
    n, Hq, d = q.shape
    Hkv = k.shape[1]
    grp = Hq // Hkv
    out = np.empty_like(q)
    for h in range(Hq):
        kh, vh = k[:, h // grp, :], v[:, h // grp, :]
        s = (q[:, h, :] @ kh.T) / np.sqrt(float(d))
        s = np.where(allowed, s, NEG_INF)
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=1, keepdims=True)
        out[:, h, :] = p @ vh
    return out


def confidence(logits: np.ndarray, mask_id: int):
    """Per row: prediction and softmax max-probability with the mask token excluded (Sec. 3.4,
    "confidence-aware parallel decoding").  pred = argmax (lowest id on an exact tie);
    conf = max softmax = 1 / sum exp(l - l_max).  Also returns the top-2 probability margin."""
    l = np.array(logits, dtype=np.float64, copy=True)
    l[:, mask_id] = NEG_INF
    pred = np.argmax(l, axis=1)
    lmax = l[np.arange(l.shape[0]), pred]
    z = np.exp(l - lmax[:, None]).sum(axis=1)
    conf = 1.0 / z
    l2 = l.copy()
    l2[np.arange(l.shape[0]), pred] = NEG_INF
    second = np.exp(l2.max(axis=1) - lmax) / z
    return pred.astype(np.int64), conf, conf - second


def select_unmask(conf: np.ndarray, masked: np.ndarray, rule: str, threshold: float = 0.9, k: int = 8) -> np.ndarray:
    """Which masked positions are revealed in this step (Sec. 3.4; Sec. 4.5 "Decoding threshold").

    threshold rule: every masked i with conf_i > tau (strict, so that tau = 1.0 reveals one token
    per step as Sec. 4.5 reports); if none qualifies, the single masked position of highest
    confidence.  top-k rule: the min(k, #masked) masked positions of highest confidence.
    Ties go to the lowest position index."""
    masked = np.asarray(masked, dtype=bool)
    sel = np.zeros_like(masked)
    idx = np.flatnonzero(masked)
    if idx.size == 0:
        return sel
    order = sorted(idx.tolist(), key=lambda i: (-conf[i], i))
    if rule == THRESHOLD:
        hit = [i for i in idx.tolist() if conf[i] > threshold]
        chosen = hit if hit else order[:1]
    elif rule == TOPK:
        chosen = order[:min(k, len(order))]
    else:
        raise ValueError(rule)
    sel[chosen] = True
    return sel


# ----------------------------------------------------------------------------------------------
# the model
# ----------------------------------------------------------------------------------------------
class Oracle:
    """One request at batch size one.

    `shape` needs attributes n_layers, hidden, n_q_heads, n_kv_heads, head_dim, intermediate, vocab,
    mask_id, rms_eps, rope_theta, tie_embeddings.  `weights` is a dict of numpy storage arrays:
    'embed', 'lm_head'/'s_lm_head' (None if tied), 'g_final', 'layers' = list of dicts with
    wq wk wv wo w_gate w_up w_down ([out, in]), optional s_* per-output-channel scales, optional
    bq bk bv, g_attn, g_mlp.
    """

    def __init__(self, shape, weights, ftype=np.float64, act_fp8: bool = False):
        """act_fp8: the input rows of the four layer projections (QKV, O, gate/up, down) pass through
        quantize_rows_e4m3 -- W8A8 when the weights are FP8 as well.  The LM head keeps unquantised inputs."""
        self.s = shape
        self.w = weights
        self.ft = ftype
        self.act_fp8 = act_fp8
        self.reset()

    def _act(self, a: np.ndarray) -> np.ndarray:
        return quantize_rows_e4m3(a).astype(self.ft) if self.act_fp8 else a

    # -- state ---------------------------------------------------------------------------------
    def reset(self):
        s = self.s
        self.K = [np.zeros((0, s.n_kv_heads, s.head_dim), dtype=self.ft) for _ in range(s.n_layers)]
        self.V = [np.zeros((0, s.n_kv_heads, s.head_dim), dtype=self.ft) for _ in range(s.n_layers)]
        self.cache_len = 0
        self.block_tokens = None
        self.masked = None
        self.step_index = 0

    # -- weights -------------------------------------------------------------------------------
    def _lin(self, layer: int, name: str) -> np.ndarray:
        lw = self.w["layers"][layer]
        w = to_f64(lw[name])
        sc = lw.get({"wq": "s_q", "wk": "s_k", "wv": "s_v", "wo": "s_o", "w_gate": "s_gate",
                     "w_up": "s_up", "w_down": "s_down"}[name])
        if sc is not None:
            w = w * to_f64(sc)[:, None]
        return w.astype(self.ft)

    def _vec(self, a):
        return None if a is None else to_f64(a).astype(self.ft)

    def embed_tokens(self, tokens) -> np.ndarray:
        tokens = np.asarray(tokens, dtype=np.int64)
        return to_f64(self.w["embed"][tokens]).astype(self.ft)

    # -- forward over n new rows against the cache -------------------------------------------
    def forward_rows(self, x: np.ndarray, mode: str, update_cache: bool) -> np.ndarray:
        """Final hidden states (before the last norm) of n new rows at positions L .. L+n-1.

        Keys allowed for row i: every cached key (M_N2C; Alg. 1 draft/verify both read the whole
        KV cache) plus, among the n new rows, all of them in BIDIR mode (Alg. 1 draft mask,
        A_ij = 1) or rows j <= i in CAUSAL mode (Alg. 1 verify mask, A_ij = 1[i >= j]; M_C2C).
        The cache is appended with the new rows' post-rotary K and V only if update_cache
        (Alg. 1: draft = "no cache update", verify/prefill = "update cache")."""
        n = x.shape[0]
        L = self.cache_len
        if mode == CAUSAL:
            among = np.tril(np.ones((n, n), dtype=bool))
        elif mode == BIDIR:
            among = np.ones((n, n), dtype=bool)
        else:
            raise ValueError(mode)
        h, k_new, v_new = self.forward_rows_masked(x, among, np.arange(L, L + n))
        if update_cache:
            self.append_cache(k_new, v_new, np.arange(n))
        return h

    def forward_rows_masked(self, x: np.ndarray, among: np.ndarray, pos: np.ndarray):
        """n new rows against the cache under an explicit mask among themselves: row i reads every cached key and the
        new rows j with among[i, j]; pos[i] is row i's position id (rotary).  The cache is not touched.
        Returns (final hidden states, per-layer post-rotary K of the new rows, per-layer V)."""
        s = self.s
        n = x.shape[0]
        L = self.cache_len
        allowed = np.ones((n, L + n), dtype=bool)
        allowed[:, L:] = among
        pos = np.asarray(pos)
        k_new, v_new = [], []
        h = np.array(x, dtype=self.ft, copy=True)
        for l in range(s.n_layers):
            lw = self.w["layers"][l]
            a = self._act(rmsnorm(h, self._vec(lw["g_attn"]), s.rms_eps))
            q = a @ self._lin(l, "wq").T
            k = a @ self._lin(l, "wk").T
            v = a @ self._lin(l, "wv").T
            if lw.get("bq") is not None:
                q = q + self._vec(lw["bq"])
                k = k + self._vec(lw["bk"])
                v = v + self._vec(lw["bv"])
            q = rope(q.reshape(n, s.n_q_heads, s.head_dim), pos, s.rope_theta)
            k = rope(k.reshape(n, s.n_kv_heads, s.head_dim), pos, s.rope_theta)
            v = v.reshape(n, s.n_kv_heads, s.head_dim)
            k_all = np.concatenate([self.K[l], k], axis=0)
            v_all = np.concatenate([self.V[l], v], axis=0)
            o = self._act(attend(q, k_all, v_all, allowed).reshape(n, s.n_q_heads * s.head_dim))
            h = h + o @ self._lin(l, "wo").T
            m = self._act(rmsnorm(h, self._vec(lw["g_mlp"]), s.rms_eps))
            act = self._act(silu(m @ self._lin(l, "w_gate").T) * (m @ self._lin(l, "w_up").T))
            h = h + act @ self._lin(l, "w_down").T
            k_new.append(k)
            v_new.append(v)
        return h, k_new, v_new

    def append_cache(self, k_new, v_new, rows):
        """The cache gains, in the order given, the K / V of `rows` of a forward_rows_masked result."""
        rows = np.asarray(rows, dtype=np.int64)
        for l in range(self.s.n_layers):
            self.K[l] = np.concatenate([self.K[l], k_new[l][rows]], axis=0)
            self.V[l] = np.concatenate([self.V[l], v_new[l][rows]], axis=0)
        self.cache_len += len(rows)

    def logits_of(self, h: np.ndarray, chunk: int = 16384) -> np.ndarray:
        """RMSNorm(h; g_final) E_out^T, E_out = the embedding table when tied."""
        s = self.s
        a = rmsnorm(h, self._vec(self.w["g_final"]), s.rms_eps)
        table = self.w["embed"] if self.w.get("lm_head") is None else self.w["lm_head"]
        sc = None if self.w.get("lm_head") is None else self.w.get("s_lm_head")
        out = np.empty((h.shape[0], s.vocab), dtype=self.ft)
        for r0 in range(0, s.vocab, chunk):
            r1 = min(s.vocab, r0 + chunk)
            wt = to_f64(table[r0:r1])
            if sc is not None:
                wt = wt * to_f64(sc[r0:r1])[:, None]
            out[:, r0:r1] = a @ wt.astype(self.ft).T
        return out

    # -- the request-level operations (same names as the C-ABI) ----------------------------------
    def prefill(self, embeds=None, tokens=None, want_logits: bool = True):
        """Causal forward over [embeds ; tokens] appended to the cache (Alg. 1, "Prefill (causal
        attention)").  Returns the last row's logits (the AR seed of Sec. 3.4) or None."""
        rows = []
        if embeds is not None and len(embeds):
            rows.append(to_f64(np.asarray(embeds)).astype(self.ft))
        if tokens is not None and len(tokens):
            rows.append(self.embed_tokens(tokens))
        if not rows:
            return None
        h = self.forward_rows(np.concatenate(rows, axis=0), CAUSAL, update_cache=True)
        return self.logits_of(h[-1:])[0] if want_logits else None

    def block_begin(self, block_size: int, init_tokens=None):
        """Start a block: B positions at L .. L+B-1.  Positions whose init token is the mask id
        (all of them by default) are masked; any other init token is a given, already revealed
        token (this is how an AR-seeded first token, Sec. 3.4, enters)."""
        s = self.s
        if init_tokens is None:
            toks = np.full(block_size, s.mask_id, dtype=np.int64)
        else:
            toks = np.asarray(init_tokens, dtype=np.int64).copy()
            assert toks.shape == (block_size,)
        self.block_tokens = toks
        self.masked = toks == s.mask_id
        self.step_index = 0

    def block_forward(self) -> np.ndarray:
        """Logits [B, vocab] of the current block in denoise mode; the cache is untouched."""
        h = self.forward_rows(self.embed_tokens(self.block_tokens), BIDIR, update_cache=False)
        return self.logits_of(h)

    def block_step(self, rule: str = THRESHOLD, threshold: float = 0.9, k: int = 8, pred_shift: int = 0):
        """One denoise step (Sec. 3.4): forward, confidence, selection, reveal.

        pred_shift = 0: row i predicts position i.  pred_shift = 1 (Appendix B, Alg. 1 "shift-by-one"): row i-1
        predicts position i; position 0 has no predictor, it must already hold a given token (the AR seed of Sec. 3.4
        "causal context decoding").  `conf` / `pred` in the record are per ROW; `pos_conf` / `pos_pred` are what
        the selection used per POSITION.

        Returns dict(logits, conf, pred, margin, pos_conf, pos_pred, unmask, block_tokens, n_unmasked, n_remaining,
        masked_before)."""
        assert pred_shift in (0, 1)
        logits = self.block_forward()
        pred, conf, margin = confidence(logits, self.s.mask_id)
        if pred_shift:
            assert not self.masked[0], "with shift-by-one the first position of the block must be given"
            pos_pred = np.concatenate([[-1], pred[:-1]])
            pos_conf = np.concatenate([[NEG_INF], conf[:-1]])
        else:
            pos_pred, pos_conf = pred, conf
        before = self.masked.copy()
        sel = select_unmask(pos_conf, self.masked, rule, threshold, k)
        self.block_tokens[sel] = pos_pred[sel]
        self.masked = self.masked & ~sel
        self.step_index += 1
        return dict(logits=logits, conf=conf, pred=pred, margin=margin, pos_conf=pos_conf, pos_pred=pos_pred, unmask=sel,
                    block_tokens=self.block_tokens.copy(), n_unmasked=int(sel.sum()),
                    n_remaining=int(self.masked.sum()), masked_before=before)

    def commit_block(self, want_logits: bool = True, all_rows: bool = False):
        """Causal pass over the finished block with cache update (Alg. 1 verify pass; clean context
        is token-causal, Sec. 3.3 M_C2C).  K/V computed during denoise passes are never stored.
        Returns the last row's logits, or with all_rows the logits of every block row [B, vocab]
        (row i = the autoregressive distribution of the token after block position i)."""
        assert self.block_tokens is not None and not self.masked.any()
        h = self.forward_rows(self.embed_tokens(self.block_tokens), CAUSAL, update_cache=True)
        self.block_tokens, self.masked = None, None
        if all_rows:
            return self.logits_of(h)
        return self.logits_of(h[-1:])[0] if want_logits else None

    def truncate(self, new_len: int):
        """Drop the cache entries of positions >= new_len (Alg. 1 "Crop")."""
        assert self.block_tokens is None and 0 <= new_len <= self.cache_len
        for l in range(self.s.n_layers):
            self.K[l] = self.K[l][:new_len]
            self.V[l] = self.V[l][:new_len]
        self.cache_len = new_len

    def decode_block(self, block_size: int, rule: str, threshold: float = 0.9, k: int = 8, init_tokens=None,
                     pred_shift: int = 0):
        """Denoise one block to completion and commit it; returns the list of step records."""
        self.block_begin(block_size, init_tokens)
        steps = []
        while self.masked.any():
            steps.append(self.block_step(rule, threshold, k, pred_shift))
            assert steps[-1]["n_unmasked"] >= 1 and len(steps) <= block_size
        next_logits = self.commit_block()
        return steps, next_logits

    def decode_block_seeded(self, block_size: int, seed_token: int, rule: str, threshold: float = 0.9, k: int = 8):
        """A block decoded the paper's way (Sec. 3.4 "causal context decoding"; Alg. 1's block layout): the first
        position holds the AR seed, the other B-1 are masks filled under shift-by-one; then the causal commit, whose
        last row's argmax (mask token excluded) is the next block's seed.  Returns (block tokens, steps, next seed)."""
        init = np.full(block_size, self.s.mask_id, dtype=np.int64)
        init[0] = seed_token
        self.block_begin(block_size, init)
        steps = []
        while self.masked.any():
            steps.append(self.block_step(rule, threshold, k, pred_shift=1))
            assert steps[-1]["n_unmasked"] >= 1 and len(steps) <= block_size - 1
        tokens = self.block_tokens.copy()
        next_logits = self.commit_block()
        return tokens, steps, int(confidence(next_logits[None, :], self.s.mask_id)[0][0])

    def spec_block(self, block_size: int, seed_token: int):
        """One iteration of linear self-speculative decoding (Sec. 3.4; Appendix B, Alg. 1), in its notation:

        d = [x_n, M, ..., M]; draft pass (denoise attention, no cache update): d_i <- argmax of row i-1 for the mask
        positions i; verify pass (causal, cache updated with all B rows): a_i = argmax of row i; accept
        k = 1 + min{ j in [0, B-2] : a_j != d_{j+1} } (no mismatch: k = B, the reading taken where Alg. 1 leaves the
        minimum of an empty set undefined); the sequence gains a_0 .. a_{k-1}; the cache is cropped to the entries of
        d_0 .. d_{k-1}.  a_{k-1} is the next iteration's x_n.  Argmax excludes the mask token.
        Returns dict(draft, a, accepted, new_tokens, next_token)."""
        B = block_size
        L0 = self.cache_len
        init = np.full(B, self.s.mask_id, dtype=np.int64)
        init[0] = seed_token
        self.block_begin(B, init)
        if B > 1:
            rec = self.block_step(THRESHOLD, NEG_INF, 0, pred_shift=1)      # every mask position filled in one pass
            assert rec["n_remaining"] == 0
        d = self.block_tokens.copy()
        a = confidence(self.commit_block(all_rows=True), self.s.mask_id)[0]
        k = accept_length(a, d)
        self.truncate(L0 + k)
        return dict(draft=d, a=a, accepted=k, new_tokens=a[:k].copy(), next_token=int(a[k - 1]))

    # -- quadratic self-speculative decoding (Appendix B, Alg. 2) -------------------------------------
    def quad_first_draft(self, block_size: int, last_logits: np.ndarray) -> np.ndarray:
        """Alg. 2 step 1 in cached form.  The prompt is in the cache (its rows ran causally, as the step-1 mask
        prescribes for them) and `last_logits` is its last row's output; B mask tokens follow, each reading the whole
        prompt and every mask token.  d_i = argmax h_{L-1+i}: d_0 comes from the prompt's last row, d_1 .. d_{B-1}
        from the first B-1 mask rows.  The cache keeps the prompt only.  Argmax excludes the mask token."""
        B = block_size
        d0 = confidence(np.asarray(last_logits)[None, :], self.s.mask_id)[0][0]
        x = self.embed_tokens(np.full(B, self.s.mask_id, dtype=np.int64))
        h = self.forward_rows(x, BIDIR, update_cache=False)
        pred = confidence(self.logits_of(h), self.s.mask_id)[0]
        return np.concatenate([[d0], pred[:B - 1]]).astype(np.int64)

    def quad_step(self, d, chain: bool = False):
        """One iteration of Alg. 2's verify + propose loop on the draft block d (B tokens; the cache holds the prompt and
        the s tokens accepted so far, cache_len = L + s).

        Input q = B groups [d_i, M^B]; position ids cache_len + i + j for entry j of group i; mask = quad_mask; one
        forward, no cache update; P_{i,j} = argmax (mask token excluded) of entry j of group i; acceptance and the next
        draft by quad_accept; the cache gains the K / V of the first tokens of groups 0 .. k-1 (of the forward's
        entries only every (B+1)-th belongs to a draft token, and of those only the accepted ones are part of the
        sequence).  Returns dict(logits [B(B+1), vocab] in the order of q, P [B, B+1], accepted, new_tokens,
        next_draft)."""
        d = np.asarray(d, dtype=np.int64)
        B = len(d)
        q = quad_input(d, self.s.mask_id)
        pos = quad_positions(self.cache_len, B)
        h, k_new, v_new = self.forward_rows_masked(self.embed_tokens(q), quad_mask(B, chain), pos)
        logits = self.logits_of(h)
        P = confidence(logits, self.s.mask_id)[0].reshape(B, B + 1)
        k, d_next = quad_accept(P, d)
        self.append_cache(k_new, v_new, np.arange(k) * (B + 1))
        return dict(logits=logits, P=P, accepted=k, new_tokens=d[:k].copy(), next_draft=d_next)

    # -- brute force: no cache, explicit [T, T] mask ----------------------------------------------
    def forward_dense(self, x: np.ndarray, allowed: np.ndarray, positions=None) -> np.ndarray:
        """Logits of T rows recomputed from scratch under an explicit boolean mask allowed[i, j]
        (row i may read key j).  Independent of the cached path: no cache, no modes; every score is
        formed one (row, key, head) at a time."""
        s = self.s
        T = x.shape[0]
        pos = np.arange(T) if positions is None else np.asarray(positions)
        h = np.array(x, dtype=np.float64, copy=True)
        grp = s.n_q_heads // s.n_kv_heads
        d = s.head_dim
        for l in range(s.n_layers):
            lw = self.w["layers"][l]
            a = rmsnorm(h, to_f64(lw["g_attn"]), s.rms_eps)
            q = a @ self._lin(l, "wq").T.astype(np.float64)
            k = a @ self._lin(l, "wk").T.astype(np.float64)
            v = a @ self._lin(l, "wv").T.astype(np.float64)
            if lw.get("bq") is not None:
                q, k, v = q + to_f64(lw["bq"]), k + to_f64(lw["bk"]), v + to_f64(lw["bv"])
            q = rope(q.reshape(T, s.n_q_heads, d), pos, s.rope_theta)
            k = rope(k.reshape(T, s.n_kv_heads, d), pos, s.rope_theta)
            v = v.reshape(T, s.n_kv_heads, d)
            o = np.zeros((T, s.n_q_heads, d))
            for i in range(T):
                keys = [j for j in range(T) if allowed[i, j]]
                for hq in range(s.n_q_heads):
                    hk = hq // grp
                    sc = np.array([np.dot(q[i, hq], k[j, hk]) / np.sqrt(d) for j in keys])
                    e = np.exp(sc - sc.max())
                    p = e / e.sum()
                    for pj, j in zip(p, keys):
                        o[i, hq] += pj * v[j, hk]
            h = h + o.reshape(T, -1) @ self._lin(l, "wo").T.astype(np.float64)
            m = rmsnorm(h, to_f64(lw["g_mlp"]), s.rms_eps)
            act = silu(m @ self._lin(l, "w_gate").T.astype(np.float64)) * (m @ self._lin(l, "w_up").T.astype(np.float64))
            h = h + act @ self._lin(l, "w_down").T.astype(np.float64)
        return np.asarray(self.logits_of(h.astype(self.ft)), dtype=np.float64)


def accept_length(a, d) -> int:
    """Alg. 1 "Accept: left-to-right comparison": k = min{ j in [0, B-2] : a_j != d_{j+1} }, then k + 1; with no
    mismatch the minimum is taken as B-1 (all B accepted)."""
    B = len(d)
    mism = [j for j in range(0, B - 1) if a[j] != d[j + 1]]
    return (mism[0] if mism else B - 1) + 1


def verify_mask(L: int, B: int) -> np.ndarray:
    """Boolean [B, L+B] mask of Alg. 1's verify step: the whole cache, and block keys j <= i (A_ij = 1[i >= j])."""
    m = np.ones((B, L + B), dtype=bool)
    m[:, L:] = np.tril(np.ones((B, B), dtype=bool))
    return m


def draft_mask(L: int, B: int) -> np.ndarray:
    """Alg. 2 step-1 mask over [prompt ; mask block]: prompt rows causal, block rows see everything."""
    T = L + B
    m = np.tril(np.ones((T, T), dtype=bool))
    m[L:, :] = True
    return m


def causal_mask(T: int) -> np.ndarray:
    return np.tril(np.ones((T, T), dtype=bool))


# -- Appendix B, Alg. 2 ("Quadratic Speculative Block-Causal Decoding") ---------------------------------------------
def quad_input(d, mask_id: int) -> np.ndarray:
    """q = [d_0, M^B, d_1, M^B, ..., d_{B-1}, M^B]: B groups of B+1 tokens, group i = the draft token d_i followed
    by B mask tokens.  Entry j of group i has index i (B+1) + j."""
    B = len(d)
    q = np.full(B * (B + 1), mask_id, dtype=np.int64)
    q[::B + 1] = np.asarray(d, dtype=np.int64)
    return q


def quad_positions(s_abs: int, B: int) -> np.ndarray:
    """Position ids: group i covers [s+i, s+i+1, ..., s+i+B] ("if accepted up to d_i, generate the next B tokens");
    s_abs = the absolute position of d_0, i.e. prompt length + accepted tokens."""
    return np.array([s_abs + i + j for i in range(B) for j in range(B + 1)], dtype=np.int64)


def quad_mask(B: int, chain: bool = False) -> np.ndarray:
    """Boolean [B(B+1), B(B+1)] mask among the entries of q (rule (a), "all tokens attend to the entire KV cache",
    is outside this matrix):
      (b) the first token of group i reads the first tokens of groups <= i;
      (c) a non-first token of group i reads every token of group i;
      (d) nothing else: no attention across groups for non-first tokens.
    chain=True is the other reading of (d) (non-first tokens are not READ across groups): a non-first token of group i
    also reads the first tokens of groups < i, the draft tokens its position ids assume accepted."""
    n = B * (B + 1)
    m = np.zeros((n, n), dtype=bool)
    for i in range(B):
        first = i * (B + 1)
        for i2 in range(i + 1):
            m[first, i2 * (B + 1)] = True                       # (b)
        for j in range(1, B + 1):
            m[first + j, first:first + B + 1] = True            # (c)
            if chain:
                for i2 in range(i):
                    m[first + j, i2 * (B + 1)] = True
    return m


def quad_accept(P, d):
    """Alg. 2's verify loop: k = 1, next draft = P_{0,1:B}; while k < B and P_{k-1,0} = d_k: next draft = P_{k,1:B},
    k += 1.  (P_{i,0}, the first token of group i, is the autoregressive prediction for the position after d_i;
    P_{i,1..B} are the mask tokens' own predictions for the B positions after d_i.)  Returns (k, next draft)."""
    P = np.asarray(P)
    B = len(d)
    k = 1
    d_next = P[0, 1:B + 1].copy()
    while k < B and P[k - 1, 0] == d[k]:
        d_next = P[k, 1:B + 1].copy()
        k += 1
    return k, d_next

