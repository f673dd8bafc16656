"""CPU oracle for token-pruned prefill and decode with an Aux Cache.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of the method
(Section 3.1 background, Section 3.2 progressive token pruning with Eq. 1, and the
Aux Cache paragraphs) that the CUDA library is checked against.  It is imported by
the tests, by the smoke check and by the CPU-baseline leg of the benchmark, and by
nothing else; it shares no code with the CUDA path.

Arithmetic: numpy float64 throughout.  Inputs (weights, ids, hidden states) arrive
as arrays of any float dtype and are widened to float64 where they are used.  No
blocking, fusion or reordering: every attention matrix is formed explicitly.

Readings of points the paper leaves open (all listed in the design document):
  * Eq. 1: query = the last token, key = token i, i.e. the LAST ROW of the usual
    [query, key] probability matrix, averaged over heads.
  * The score of layer e-1 selects the set that enters layer e (Section 3.2: the
    score s^l decides what the following layer still sees); the cut sits between attention (+ output
    projection + residual) and the MLP of layer e-1, so that MLP already runs on
    the kept rows only and the Aux Cache of layer e-1 holds post-attention,
    pre-MLP hidden states.  The literal alternative (cut after the whole layer, Aux
    Cache = the layer's output) is the aux_point="post_layer" switch; both give the
    kept and revived tokens identical values downstream (pinned in the tests).
  * The keep fraction is cumulative, of the ORIGINAL token count, in integer basis
    points; count = ceil(bp*N/10000) clamped to [1, rows present]; count-based
    top-k; ties go to the lower position; the last token is never pruned; kept
    rows stay in ascending position order; RoPE uses original positions.
  * Decode-step selection semantics (which set is attended, percentile base p+1,
    Aux eviction on revival) are this oracle's own definition: PARITY UNPINNED by
    the paper for those choices; only invariants constrain them.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------- layer maths
def f64(a) -> np.ndarray:
    return np.asarray(a, dtype=F64)


def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """Root-mean-square norm with gain (Llama 2 layer norm; Section 4 names the model)."""
    x = f64(x)
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * f64(g)


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, half-split pairing (i, i + dh/2), angle = pos * theta^(-2i/dh).

    x: [n, H, dh]; pos: [n] original token positions.
    """
    x = f64(x)
    dh = x.shape[-1]
    half = dh // 2
    inv_freq = F64(theta) ** (-2.0 * np.arange(half, dtype=F64) / dh)
    ang = f64(pos)[:, None] * inv_freq[None, :]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def attention_probs(qh: np.ndarray, kh: np.ndarray, qpos: np.ndarray, kpos: np.ndarray) -> np.ndarray:
    """Explicit attention probabilities A[i, j] of ONE head: query row i attending to key row j.

    qh: [nq, dh], kh: [nk, dh] (both already rotated).  Key j is visible to query i iff
    kpos[j] <= qpos[i] (causal).  Softmax over j with scale 1/sqrt(dh).
    """
    dh = qh.shape[-1]
    logits = (f64(qh) @ f64(kh).T) / math.sqrt(dh)
    visible = np.asarray(kpos)[None, :] <= np.asarray(qpos)[:, None]
    logits = np.where(visible, logits, -np.inf)
    logits = logits - np.max(logits, axis=-1, keepdims=True)
    e = np.exp(logits)
    return e / np.sum(e, axis=-1, keepdims=True)


def attend(q: np.ndarray, k: np.ndarray, v: np.ndarray, qpos: np.ndarray, kpos: np.ndarray,
           score_row: int) -> Tuple[np.ndarray, np.ndarray]:
    """Multi-head attention output and the importance score of Eq. 1.

    q: [nq, H, dh]; k, v: [nk, Hkv, dh] with Hkv dividing H.  With Hkv < H (grouped-query attention, the
    layout of the 7B-class models with fewer key/value heads than query heads) query head h reads
    key/value head h // (H // Hkv).  Returns (o [nq, H*dh], s [nk]) where
    s_j = (1/H) * sum_h A_h[score_row, j]: the probabilities with which the token whose
    successor is being predicted attends to token j, averaged over the H query heads.
    """
    nq, H, dh = q.shape
    Hkv = k.shape[1]
    assert H % Hkv == 0 and v.shape[1] == Hkv
    group = H // Hkv
    o = np.zeros((nq, H, dh), dtype=F64)
    s = np.zeros(k.shape[0], dtype=F64)
    for h in range(H):
        A = attention_probs(q[:, h, :], k[:, h // group, :], qpos, kpos)
        o[:, h, :] = A @ f64(v[:, h // group, :])
        s += A[score_row, :]
    return o.reshape(nq, H * dh), s / H


def keep_count(n_total: int, keep_bp: int, n_present: int) -> int:
    """ceil(keep_bp/10000 * n_total) in integers, clamped to [1, n_present]."""
    c = (int(n_total) * int(keep_bp) + 9999) // 10000
    return max(1, min(int(n_present), c))


def select_top(scores: np.ndarray, n_keep: int, forced: int) -> Tuple[np.ndarray, np.ndarray]:
    """Top-percentile selection (Section 3.2) as a count-based top-k.

    Keeps the ``n_keep`` candidates with the largest score; candidate ``forced`` (the
    token being predicted from) is always kept and counts toward ``n_keep``; among equal
    scores the lower index wins.  Returns (kept ascending, dropped ascending) as indices
    into ``scores``.
    """
    s = np.asarray(scores)
    n = s.shape[0]
    if forced < 0:
        forced += n
    assert 1 <= n_keep <= n
    others = [i for i in range(n) if i != forced]
    others.sort(key=lambda i: (-float(s[i]), i))
    kept = sorted([forced] + others[: n_keep - 1])
    dropped = sorted(others[n_keep - 1:])
    return np.asarray(kept, dtype=np.int64), np.asarray(dropped, dtype=np.int64)


def select_ties_kept(scores: np.ndarray, n_keep: int, forced: int) -> Tuple[np.ndarray, np.ndarray]:
    """The selection of Section 3.2 read as a THRESHOLD at the same percentile the count form uses.

    tau = the n_keep-th largest score among the candidates, the forced candidate (the token being predicted
    from) counting as larger than everything.  A token is pruned iff its score is smaller than tau; scores
    equal to tau are not smaller, so every tie at the threshold is kept and the number of kept tokens
    (>= n_keep) depends on the data.  Without ties at tau this is exactly `select_top`.
    Returns (kept ascending, dropped ascending).
    """
    s = np.asarray(scores)
    n = s.shape[0]
    if forced < 0:
        forced += n
    assert 1 <= n_keep <= n
    others = sorted((float(s[i]) for i in range(n) if i != forced), reverse=True)
    if n_keep == 1:
        kept = [forced]
    else:
        tau = others[n_keep - 2]                      # the forced token takes the first of the n_keep places
        kept = [i for i in range(n) if i == forced or float(s[i]) >= tau]
    drop = [i for i in range(n) if i not in set(kept)]
    return np.asarray(kept, dtype=np.int64), np.asarray(drop, dtype=np.int64)


SELECTIONS = ("count", "threshold")


def _select(selection: str, scores, n_keep: int, forced: int):
    if selection == "count":
        return select_top(scores, n_keep, forced)
    if selection == "threshold":
        return select_ties_kept(scores, n_keep, forced)
    raise ValueError(f"selection must be one of {SELECTIONS}")


# --------------------------------------------------------------------------- model pieces
def select_threshold(scores: np.ndarray, prune_bp: int) -> Tuple[np.ndarray, np.ndarray]:
    """The selection of Section 3.2 read as a threshold: a token is pruned if its score is smaller than
    the prune_bp/100-th percentile of the scores; the last token is never pruned.

    Percentile = the order statistic with index floor((n-1) * prune_bp / 10000) from below (the "lower"
    definition: no interpolation, so the threshold is one of the scores and comparisons are exact in
    the scores' own precision).  Ties at the threshold are all kept: the count depends on the data.
    Returns (kept, dropped) row indices, ascending.
    """
    s = np.asarray(scores)
    n = s.shape[0]
    if n == 0:
        return np.zeros(0, dtype=np.int64), np.zeros(0, dtype=np.int64)
    if not 0 <= prune_bp <= 9999:
        raise ValueError("prune_bp must be in 0..9999")
    tau = np.sort(s)[((n - 1) * int(prune_bp)) // 10000]
    keep = np.asarray([i for i in range(n) if s[i] >= tau or i == n - 1], dtype=np.int64)
    drop = np.asarray([i for i in range(n) if not (s[i] >= tau or i == n - 1)], dtype=np.int64)
    return keep, drop


# --------------------------------------------------------------------------- fp8 projections
# Optional 8-bit mode of the four projections of a layer (QKV, output, gate/up, down): both operands of the
# product are e4m3 numbers (4 exponent bits, 3 mantissa bits, largest finite value 448, no infinities) times
# a scale.  Weights arrive already rounded (a per-matrix scale folded in by whoever made them: the oracle is
# handed the de-quantised values).  Activations are quantised per ROW on the way into the product, in the
# arithmetic the CUDA path uses for the decision (float32): scale = max|x| / 448 (1 for an all-zero row),
# code = round-to-nearest-even of x / scale onto the e4m3 grid.  The product itself is exact (float64) here.
E4M3_MAX = 448.0


def round_e4m3(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest e4m3 number (ties to even), saturating at +-448.  Written out on
    the bit level: 3 mantissa bits above 2^-6 (normal numbers), a fixed step of 2^-9 below (subnormals)."""
    x = np.asarray(x, dtype=np.float32)
    a = np.minimum(np.abs(x).astype(np.float64), E4M3_MAX)
    e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.maximum(e, -6.0)                               # below 2^-6 the grid no longer refines
    step = np.exp2(e - 3.0)                               # 8 steps per binade
    q = np.round(a / step) * step                         # numpy rounds halves to even
    q = np.minimum(q, E4M3_MAX)
    return (np.sign(x) * q).astype(np.float32)


def quant_rows_e4m3(x: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Per-row e4m3 quantisation of activations.  Returns (codes as float32 values on the e4m3 grid,
    scale per row as float32); the de-quantised activation is codes * scale."""
    x32 = np.asarray(x, dtype=np.float32)
    amax = np.max(np.abs(x32), axis=-1, keepdims=True)
    scale = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
    codes = round_e4m3((x32 / scale).astype(np.float32))
    return codes, scale[..., 0]


def _bf16_round(x: np.ndarray) -> np.ndarray:
    """Nearest bfloat16 (ties to even) of every element, as float32."""
    u = np.ascontiguousarray(np.asarray(x, dtype=np.float32)).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) & np.uint32(0xFFFF0000)).view(np.float32)


def _linear(cfg, x, w):
    """x @ w^T.  With cfg.fp8 the activation rows are quantised to e4m3 first (see above), from their
    bfloat16 values: that is what the CUDA path holds when it takes the rounding decisions."""
    if getattr(cfg, "fp8", False):
        codes, scale = quant_rows_e4m3(_bf16_round(x))
        x = f64(codes) * f64(scale)[..., None]
    return f64(x) @ f64(w).T


def kv_heads(cfg) -> int:
    """Key/value heads of the shape (grouped-query attention when fewer than the query heads)."""
    return int(getattr(cfg, "n_kv_heads", 0) or cfg.n_heads)


def _layer_qkv(cfg, lw, x, pos):
    """Pre-norm, QKV projection, head split, RoPE on q and k.  w_qkv = [q rows | k rows | v rows] with
    H*dh, Hkv*dh and Hkv*dh rows."""
    H, dh, d = cfg.n_heads, cfg.head_dim, cfg.d_model
    Hkv = kv_heads(cfg)
    dkv = Hkv * dh
    h = rmsnorm(x, lw["g_attn"], cfg.rms_eps)
    qkv = _linear(cfg, h, lw["w_qkv"])
    n = x.shape[0]
    q = rope(qkv[:, :d].reshape(n, H, dh), pos, cfg.rope_theta)
    k = rope(qkv[:, d:d + dkv].reshape(n, Hkv, dh), pos, cfg.rope_theta)
    v = qkv[:, d + dkv:].reshape(n, Hkv, dh)
    return q, k, v


def _o_proj(cfg, o, lw):
    """Output projection of the concatenated heads."""
    return _linear(cfg, o, lw["w_o"])


def mlp(cfg, lw, x):
    """SwiGLU MLP of a pre-norm block: (silu(h Wg^T) * (h Wu^T)) Wd^T, h = rmsnorm(x)."""
    h = rmsnorm(x, lw["g_mlp"], cfg.rms_eps)
    return _linear(cfg, silu(_linear(cfg, h, lw["w_gate"])) * _linear(cfg, h, lw["w_up"]), lw["w_down"])


def lm_head(cfg, W, x_row):
    return rmsnorm(x_row, W["g_final"], cfg.rms_eps) @ f64(W["w_lm_head"]).T


# --------------------------------------------------------------------------- caches
# Where in the scoring layer the token set is cut (Section 3.2, Aux Cache paragraph).
#   "pre_mlp":    between the attention half (attention, output projection, residual) and the MLP, so the
#                 layer's MLP already runs on the kept rows and the Aux Cache holds post-attention states;
#                 a revived token first gets the MLP of that layer.
#   "post_layer": after the whole layer, the literal wording ("stores the hidden states of those pruned
#                 tokens"): the MLP runs on every row and the Aux Cache holds the layer's output.
# The MLP is row-wise, so both give every kept or revived token the same values in every later layer.
AUX_POINTS = ("pre_mlp", "post_layer")


class LayerCache:
    """KV cache of one layer with position tags, and the Aux Cache that follows it.

    kv: position -> (k [H,dh], v [H,dh]) for every token whose KV exists at this layer.
    aux: position -> hidden state (post-attention residual stream of this layer, or the layer's
    output with aux_point "post_layer") of tokens whose KV exists here but not in the next layer's
    cache (Aux Cache paragraph).
    """

    def __init__(self):
        self.kv: Dict[int, Tuple[np.ndarray, np.ndarray]] = {}
        self.aux: Dict[int, np.ndarray] = {}

    def rows(self, positions: Sequence[int]):
        k = np.stack([self.kv[int(p)][0] for p in positions])
        v = np.stack([self.kv[int(p)][1] for p in positions])
        return k, v


class LazyState:
    """Everything one sequence carries from prefill into decode, plus per-call records."""

    def __init__(self, cfg, schedule, aux_point: str = "pre_mlp", selection: str = "count"):
        if aux_point not in AUX_POINTS:
            raise ValueError(f"aux_point must be one of {AUX_POINTS}")
        if selection not in SELECTIONS:
            raise ValueError(f"selection must be one of {SELECTIONS}")
        self.cfg = cfg
        self.aux_point = aux_point
        self.selection = selection
        self.schedule = {int(e): int(bp) for e, bp in schedule}
        self.layers = [LayerCache() for _ in range(cfg.n_layers)]
        self.n_tokens = 0                      # tokens seen so far (prompt + generated)
        # records of the latest call
        self.scores: List[np.ndarray] = []     # per layer, over that layer's candidate rows
        self.score_pos: List[np.ndarray] = []  # positions those scores refer to
        self.kept_pos: Dict[int, np.ndarray] = {}     # layer entered -> kept positions
        self.dropped_pos: Dict[int, np.ndarray] = {}  # layer entered -> dropped positions
        self.revived_pos: Dict[int, np.ndarray] = {}  # layer entered -> revived positions (decode)
        self.hidden_after_attn: List[np.ndarray] = []
        self.hidden_out: List[np.ndarray] = []
        self.rows_pos: List[np.ndarray] = []   # positions of rows computed at each layer
        self.logits: Optional[np.ndarray] = None
        self.compute_count: Dict[Tuple[int, int], int] = {}  # (layer, pos) -> times computed

    def _count(self, layer: int, positions) -> None:
        for p in positions:
            key = (layer, int(p))
            self.compute_count[key] = self.compute_count.get(key, 0) + 1

    def _reset_records(self):
        self.scores, self.score_pos = [], []
        self.kept_pos, self.dropped_pos, self.revived_pos = {}, {}, {}
        self.hidden_after_attn, self.hidden_out, self.rows_pos = [], [], []


def validate_schedule(cfg, schedule) -> None:
    prev_e, prev_bp = 0, 10000
    for e, bp in schedule:
        if not (prev_e < e < cfg.n_layers):
            raise ValueError("schedule layers must be strictly increasing in (0, n_layers)")
        if not (1 <= bp <= 10000) or bp > prev_bp:
            raise ValueError("keep fractions must be in 1..10000 and non-increasing")
        prev_e, prev_bp = e, bp


# --------------------------------------------------------------------------- prefill
def prefill(cfg, W, ids, schedule, forced_keep: Optional[Dict[int, Sequence[int]]] = None,
            keep_records: bool = True, aux_point: str = "pre_mlp", selection: str = "count") -> LazyState:
    """Token-pruned prefill of one prompt (Sections 3.1 and 3.2).

    ids: [N] token ids.  schedule: iterable of (layer_entered, cumulative keep in basis
    points of N); layer 0 always sees the whole prompt.  forced_keep: optional
    {layer_entered: kept positions} that replaces the score-based selection at that
    point (used to replay another implementation's kept sets).  aux_point: see AUX_POINTS.
    selection: "count" keeps exactly the scheduled number of tokens (ties to the lower position);
    "threshold" prunes a token iff its score is smaller than the score at that rank, so ties at the
    threshold all survive and later layers may see more rows than scheduled.
    """
    validate_schedule(cfg, schedule)
    st = LazyState(cfg, schedule, aux_point, selection)
    ids = np.asarray(ids).astype(np.int64)
    N = ids.shape[0]
    st.n_tokens = N
    x = f64(W["tok_embed"])[ids]
    pos = np.arange(N, dtype=np.int64)
    for l in range(cfg.n_layers):
        lw = W["layers"][l]
        q, k, v = _layer_qkv(cfg, lw, x, pos)
        cache = st.layers[l]
        for r, p in enumerate(pos):
            cache.kv[int(p)] = (k[r], v[r])
        st._count(l, pos)
        o, s = attend(q, k, v, pos, pos, -1)
        x = x + _o_proj(cfg, o, lw)
        if keep_records:
            st.scores.append(s)
            st.score_pos.append(pos.copy())
            st.rows_pos.append(pos.copy())
            st.hidden_after_attn.append(x.copy())
        cut = (l + 1) in st.schedule
        if cut:   # the selection itself only needs this layer's scores
            n = x.shape[0]
            if forced_keep is not None and (l + 1) in forced_keep:
                want = set(int(p) for p in forced_keep[l + 1])
                keep = np.asarray([r for r in range(n) if int(pos[r]) in want], dtype=np.int64)
                drop = np.asarray([r for r in range(n) if int(pos[r]) not in want], dtype=np.int64)
            else:
                keep, drop = _select(selection, s, keep_count(N, st.schedule[l + 1], n), n - 1)
            st.kept_pos[l + 1] = pos[keep].copy()
            st.dropped_pos[l + 1] = pos[drop].copy()
        if cut and aux_point == "pre_mlp":
            for r in drop:
                cache.aux[int(pos[r])] = x[r].copy()
            x, pos = x[keep], pos[keep]
        x = x + mlp(cfg, lw, x)
        if cut and aux_point == "post_layer":
            for r in drop:
                cache.aux[int(pos[r])] = x[r].copy()
            x, pos = x[keep], pos[keep]
        if keep_records:
            st.hidden_out.append(x.copy())
    st.logits = lm_head(cfg, W, x[-1])
    return st


# --------------------------------------------------------------------------- one layer
def layer_step(cfg, lw, x, pos, keep_pos: Optional[Sequence[int]] = None):
    """One decoder layer of the pruned prefill on given inputs (the body of the loop in `prefill`).

    x: [n, d] hidden states entering the layer, pos: [n] their positions (ascending).  If
    ``keep_pos`` is given, the cut sits after attention: rows whose position is listed go on to the
    MLP, the others are returned as the layer's Aux rows.  Returns a dict with the Eq. 1 scores, the
    post-attention hidden states of all rows, the kept positions, the output of the layer for the
    kept rows and the Aux rows / positions.
    """
    x = f64(x)
    pos = np.asarray(pos).astype(np.int64)
    q, k, v = _layer_qkv(cfg, lw, x, pos)
    o, s = attend(q, k, v, pos, pos, -1)
    y = x + _o_proj(cfg, o, lw)
    if keep_pos is not None:
        want = set(int(p) for p in keep_pos)
        keep = np.asarray([r for r in range(len(pos)) if int(pos[r]) in want], dtype=np.int64)
        drop = np.asarray([r for r in range(len(pos)) if int(pos[r]) not in want], dtype=np.int64)
    else:
        keep, drop = np.arange(len(pos)), np.zeros(0, dtype=np.int64)
    z = y[keep]
    z = z + mlp(cfg, lw, z)
    return {"scores": s, "hidden_attn": y, "k": k, "v": v, "pos_out": pos[keep], "hidden_out": z,
            "aux_rows": y[drop], "aux_pos": pos[drop]}


# --------------------------------------------------------------------------- revive
def revive(st: LazyState, layer: int, positions: Sequence[int], take: bool = False) -> np.ndarray:
    """Hidden states of pruned tokens from the Aux Cache that follows ``layer``.

    Raises KeyError if a position is not held there.  With ``take`` the entries leave
    the Aux Cache (they are about to get KV in the next layer).
    """
    aux = st.layers[layer].aux
    rows = [aux[int(p)] for p in positions]
    if take:
        for p in positions:
            del aux[int(p)]
    return np.stack(rows) if rows else np.zeros((0, st.cfg.d_model))


# --------------------------------------------------------------------------- decode
def decode_step(cfg, W, st: LazyState, token_id: int,
                forced_keep: Optional[Dict[int, Sequence[int]]] = None) -> np.ndarray:
    """One decode step with dynamic re-selection and revival (Section 3.2, Aux Cache).

    The new token sits at position p = tokens so far.  In every layer the rows "in
    flight" (the new token plus tokens revived earlier in this step) get q, k, v; their
    K/V are appended to that layer's cache; each attends, causally by position, over the
    currently selected context set T plus the new token.  At a scheduled boundary the
    new token's Eq. 1 score over T re-selects the context: selected tokens without KV in
    the next layer are revived from the Aux Cache, in-flight rows that fall out are put
    into it.  Returns the logits of the new token's row.
    """
    st._reset_records()
    p = st.n_tokens
    T = np.arange(p, dtype=np.int64)                 # selected context, ascending positions
    X: Dict[int, np.ndarray] = {p: f64(W["tok_embed"])[int(token_id)].copy()}
    for l in range(cfg.n_layers):
        lw = W["layers"][l]
        cache = st.layers[l]
        xpos = np.asarray(sorted(X.keys()), dtype=np.int64)
        x = np.stack([X[int(r)] for r in xpos])
        q, k, v = _layer_qkv(cfg, lw, x, xpos)
        for i, r in enumerate(xpos):
            assert int(r) not in cache.kv, "a token is computed at most once per layer"
            cache.kv[int(r)] = (k[i], v[i])
        st._count(l, xpos)
        ctx = np.concatenate([T, np.asarray([p], dtype=np.int64)])
        kc, vc = cache.rows(ctx)
        o, s = attend(q, kc, vc, xpos, ctx, int(np.nonzero(xpos == p)[0][0]))
        x = x + _o_proj(cfg, o, lw)
        st.scores.append(s)
        st.score_pos.append(ctx.copy())
        st.rows_pos.append(xpos.copy())
        st.hidden_after_attn.append(x.copy())
        X = {int(r): x[i] for i, r in enumerate(xpos)}
        if (l + 1) in st.schedule and st.aux_point == "post_layer":
            x = x + mlp(cfg, lw, x)                   # the cut comes after the whole layer
            st.hidden_out.append(x.copy())
            X = {int(r): x[i] for i, r in enumerate(xpos)}
        if (l + 1) in st.schedule:
            if forced_keep is not None and (l + 1) in forced_keep:
                want = set(int(t) for t in forced_keep[l + 1]) | {p}
                keep = np.asarray([i for i in range(len(ctx)) if int(ctx[i]) in want], dtype=np.int64)
            else:
                n_keep = keep_count(p + 1, st.schedule[l + 1], len(ctx))
                keep, _ = _select(st.selection, s, n_keep, len(ctx) - 1)
            sel = ctx[keep]                           # includes p
            sel_set = set(int(t) for t in sel)
            for r in list(X.keys()):                  # in flight but not selected any more
                if r not in sel_set:
                    cache.aux[r] = X.pop(r)
            nxt = st.layers[l + 1].kv
            need = [int(t) for t in sel if int(t) != p and int(t) not in nxt and int(t) not in X]
            if need:
                rows = revive(st, l, need, take=True)
                for i, r in enumerate(need):
                    X[r] = rows[i]
            st.kept_pos[l + 1] = sel.copy()
            st.revived_pos[l + 1] = np.asarray(need, dtype=np.int64)
            T = sel[sel != p]
            if st.aux_point == "post_layer":
                continue                              # revived rows already hold this layer's output
        xpos = np.asarray(sorted(X.keys()), dtype=np.int64)
        x = np.stack([X[int(r)] for r in xpos])
        x = x + mlp(cfg, lw, x)
        st.hidden_out.append(x.copy())
        X = {int(r): x[i] for i, r in enumerate(xpos)}
    st.n_tokens = p + 1
    st.logits = lm_head(cfg, W, X[p])
    return st.logits


def greedy(logits: np.ndarray) -> int:
    """Greedy next token; equal logits resolve to the lowest id."""
    return int(np.argmax(logits))


# --------------------------------------------------------------------------- single-layer prune op
def prune_op(cfg, lw, x, pos, keep_bp: int, forced_keep_rows: Optional[Sequence[int]] = None):
    """One layer's attention half followed by the cut (the single-layer pruning op).

    x: [n, d] hidden states entering the layer, pos: [n] positions.  Returns a dict with
    the Eq. 1 scores, kept / dropped row indices, the post-attention hidden states, and
    the gathered hidden / K / V / pos rows of the kept set plus the Aux rows.
    """
    x = f64(x)
    pos = np.asarray(pos).astype(np.int64)
    n = x.shape[0]
    q, k, v = _layer_qkv(cfg, lw, x, pos)
    o, s = attend(q, k, v, pos, pos, -1)
    y = x + _o_proj(cfg, o, lw)
    if forced_keep_rows is not None:
        want = set(int(r) for r in forced_keep_rows)
        keep = np.asarray([r for r in range(n) if r in want], dtype=np.int64)
        drop = np.asarray([r for r in range(n) if r not in want], dtype=np.int64)
    else:
        keep, drop = select_top(s, keep_count(n, keep_bp, n), n - 1)
    return {"scores": s, "keep": keep, "drop": drop, "hidden_attn": y, "q": q, "k": k, "v": v,
            "hidden_kept": y[keep], "k_kept": k[keep], "v_kept": v[keep], "pos_kept": pos[keep],
            "aux_rows": y[drop], "aux_pos": pos[drop]}


# --------------------------------------------------------------------------- counters
def tokens_computed_fraction(st: LazyState, n_prompt: int) -> List[float]:
    """Per layer: fraction of prompt tokens whose KV exists (cumulative token usage)."""
    return [sum(1 for p in c.kv if p < n_prompt) / float(n_prompt) for c in st.layers]
