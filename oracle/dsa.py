"""fp64 oracle for sparse (DSA) response replay over the shared latent.

Test infrastructure only; shares no code with the CUDA library (whose sparse path the GPU
tests compare against these functions).

What is computed (Sec. "GLM Attention: MLA, DSA, and IndexShare", Eq. dsa-index,
Eq. dsa-attention; Sec. "Predecessor CP-Local 2M Diagnostic", Eq. glm-global-dsa):
a response query at row t (global position P + t) scores every visible position s -- all P
prefix positions and the response positions j <= t -- with the indexer

    I_{t,s} = sum_{j=1..H_I} w_{t,j} ReLU(<qI_{t,j}, kI_s>),

keeps the k positions with the largest score (TopK over the whole logical context, not per
shard) and attends to exactly those:

    u_t = Attn(q_t, {c_s : s in TopK(I_{t,:}, k)}),

i.e. softmax over the selected positions only, with the same scores s_ts = scale <q_t, k_s>,
log-normaliser and value sum as the dense operator restricted to the selected set.  The
latent page holds the key (Dk channels) whose first Dv channels are the value.

Readings where the paper is silent:
 * visibility: causal in global coordinates, the query's own position included;
 * fewer than k visible positions: all of them are selected;
 * ties: among equal scores the LOWER global position wins (a deterministic rule is what
   Eq. glm-global-dsa asks of a cross-rank merge; which one is not stated);
 * the selection is not differentiated (TopK is piecewise constant): the backward treats the
   selected set as fixed and returns dQ over the selected keys and dK / dV for selected
   RESPONSE keys only -- the prefix stays gradient-free (Sec. "Lazy Gradient Pages").

Every array is float64; bf16 inputs arrive as uint16 bit patterns and are widened exactly.
"""
import numpy as np

from .attention import widen, _page_spans


def index_scores(qi_rows, w_rows, t_rows, ki_pool, page_table, P, pg, ki_resp):
    """Eq. dsa-index for a set of rows: I [n, P + R]; invisible response positions (j > t) are -inf.

    qi_rows [n, H_I, dI], w_rows [n, H_I]; ki_pool [pages, pg, 1, dI] (indexer-key pages, read
    through the page table like the latent pages); ki_resp [R, dI].
    """
    qi = widen(qi_rows)
    w = widen(w_rows)
    n, hi, _ = qi.shape
    R = ki_resp.shape[0]
    out = np.empty((n, P + R), dtype=np.float64)

    def block(keys):                      # keys [m, dI] -> [n, m]
        dots = np.einsum("nhd,md->nhm", qi, keys)
        return np.einsum("nh,nhm->nm", w, np.maximum(dots, 0.0))

    for p, pos, valid in _page_spans(P, pg):
        out[:, pos:pos + valid] = block(widen(ki_pool[page_table[p], :valid, 0, :]))
    out[:, P:] = block(widen(ki_resp))
    j = np.arange(R)[None, :]
    out[:, P:][j > np.asarray(t_rows)[:, None]] = -np.inf
    return out


def topk_select(scores_row, k):
    """Global positions of the k largest finite scores of one row, ascending by position.
    Ties go to the lower position.  Fewer than k visible positions: all of them."""
    s = np.asarray(scores_row, dtype=np.float64)
    visible = np.flatnonzero(np.isfinite(s) | (s == np.inf))
    if visible.size <= k:
        return visible
    # stable sort by descending score keeps the lower position first among equals
    order = visible[np.argsort(-s[visible], kind="stable")]
    return np.sort(order[:k])


def merge_shard_candidates(scores_row, shard_positions, k):
    """Eq. glm-global-dsa as a two-level selection: every shard proposes its own top-k (with global
    positions), the union is re-ranked.  Returns the same set as topk_select on the whole row."""
    cand = []
    for pos in shard_positions:
        pos = np.asarray(pos, dtype=np.int64)
        if pos.size == 0:
            continue
        local = topk_select(np.where(np.isin(np.arange(len(scores_row)), pos), scores_row, -np.inf), k)
        cand.append(local)
    cand = np.unique(np.concatenate(cand)) if cand else np.zeros(0, np.int64)
    masked = np.full(len(scores_row), -np.inf)
    masked[cand] = np.asarray(scores_row)[cand]
    return topk_select(masked, k)


def _gather_keys(sel, k_pool, page_table, P, pg, k_resp, width=None):
    """Rows of the latent (prefix through the page table, response dense) at global positions sel."""
    sel = np.asarray(sel, dtype=np.int64)
    d = k_resp.shape[-1] if width is None else width
    out = np.empty((sel.size, d), dtype=np.float64)
    pre = sel < P
    if pre.any():
        pp = sel[pre]
        out[pre] = widen(k_pool[np.asarray(page_table)[pp // pg], pp % pg, 0, :d])
    if (~pre).any():
        out[~pre] = widen(k_resp[sel[~pre] - P, 0, :d])
    return out


def sparse_forward_rows(q_rows, selections, k_pool, page_table, P, pg, k_resp, dv, scale):
    """Eq. dsa-attention for a set of rows with their selected position sets.

    q_rows [n, Dk]; selections: list of n index arrays (global positions); k_pool
    [pages, pg, 1, Dk] latent pages, k_resp [R, 1, Dk]; the value is the first dv channels.
    Returns O [n, dv], LSE [n] and the per-row probabilities (list of arrays).
    """
    q = widen(q_rows)
    n = q.shape[0]
    o = np.zeros((n, dv))
    lse = np.full(n, -np.inf)
    probs = []
    for i in range(n):
        sel = selections[i]
        if len(sel) == 0:
            probs.append(np.zeros(0))
            continue
        keys = _gather_keys(sel, k_pool, page_table, P, pg, k_resp)
        s = scale * (keys @ q[i])
        m = s.max()
        l = m + np.log(np.exp(s - m).sum())
        p = np.exp(s - l)
        lse[i] = l
        o[i] = p @ keys[:, :dv]
        probs.append(p)
    return o, lse, probs


def sparse_backward_rows(q_rows, selections, k_pool, page_table, P, pg, k_resp, dv, scale, d_o_rows):
    """Gradients of the rows with the selection held fixed: dQ [n, Dk] and the rows' contributions
    to dK_resp [R, Dk] (score path, all Dk channels, times scale) and dV_resp [R, dv] (value path) of
    the selected RESPONSE positions.  Selected prefix positions get nothing."""
    q = widen(q_rows)
    do = widen(d_o_rows)
    n, dk = q.shape
    R = k_resp.shape[0]
    o, lse, probs = sparse_forward_rows(q_rows, selections, k_pool, page_table, P, pg, k_resp, dv, scale)
    dq = np.zeros((n, dk))
    dk_resp = np.zeros((R, dk))
    dv_resp = np.zeros((R, dv))
    for i in range(n):
        sel = np.asarray(selections[i], dtype=np.int64)
        if sel.size == 0:
            continue
        keys = _gather_keys(sel, k_pool, page_table, P, pg, k_resp)
        p = probs[i]
        delta = do[i] @ o[i]
        dp = keys[:, :dv] @ do[i]
        ds = p * (dp - delta)
        dq[i] = scale * (ds @ keys)
        resp = sel >= P
        if resp.any():
            j = sel[resp] - P
            np.add.at(dk_resp, j, scale * np.outer(ds[resp], q[i]))
            np.add.at(dv_resp, j, np.outer(p[resp], do[i]))
    return o, lse, dq, dk_resp, dv_resp
