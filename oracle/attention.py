"""fp64 oracle for exact-attention response replay.

Test infrastructure only; shares no code with the CUDA library.

What is computed (Sec. "Global Full-Attention Forward Composition"):
a response query at row t (global position P + t) of query head h, with KV head
kv = h // (Hq // Hkv), sees every prefix position 0..P-1 and the response
positions j <= t.  Scores s_tj = scale * <q_th, k_j>; LSE_th = log sum_j exp(s_tj);
p_tj = exp(s_tj - LSE_th); O_th = sum_j p_tj v_j.  This is Eq. qwen-local-attn
with a single partition, i.e. the dense operator that the sharded method must
reproduce.  The prefix is read through the logical-to-physical page table
(Sec. "From Logical Shards to Physical Pages").

Backward (Sec. "Lazy Gradient Pages", Eq. qwen-dq-reduce): with upstream dO,
Delta_th = <dO_th, O_th>, dp_tj = <dO_th, v_j>, ds_tj = p_tj (dp_tj - Delta_th),
dQ_th = scale * sum_j ds_tj k_j over prefix AND response keys;
dK_j = scale * sum_{t>=j, h in group} ds_tj q_th and dV_j = sum p_tj dO_th for
RESPONSE keys only.  Prefix K/V are a stop-gradient state and get nothing.

Every array is float64.  bf16 inputs arrive as uint16 bit patterns and are
widened exactly by `widen`.
"""
import numpy as np


def widen(x):
    """Exact widening to float64.  uint16 arrays are bf16 bit patterns."""
    x = np.asarray(x)
    if x.dtype == np.uint16:
        return (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return x.astype(np.float64)


def _page_spans(P, pg):
    """(logical page, first position, valid tokens) for every prefix page."""
    p, pos = 0, 0
    while pos < P:
        n = min(pg, P - pos)
        yield p, pos, n
        p += 1
        pos += n


def _logsumexp_rows(s):
    m = s.max(axis=1)
    m_safe = np.where(np.isfinite(m), m, 0.0)
    with np.errstate(divide="ignore"):
        return m_safe + np.log(np.exp(s - m_safe[:, None]).sum(axis=1))


def scores_rows(q_rows, t_rows, kv, k_pool, page_table, P, pg, k_resp, scale):
    """s[i, j] for query rows i against all P prefix keys then all R response keys;
    response keys j > t_i are masked to -inf (causal, the query sees itself)."""
    q_rows = widen(q_rows)
    R = k_resp.shape[0]
    n = q_rows.shape[0]
    s = np.empty((n, P + R), dtype=np.float64)
    for p, pos, valid in _page_spans(P, pg):
        kp = widen(k_pool[page_table[p], :valid, kv, :])
        s[:, pos:pos + valid] = scale * (q_rows @ kp.T)
    s[:, P:] = scale * (q_rows @ widen(k_resp[:, kv, :]).T)
    j = np.arange(R)[None, :]
    s[:, P:][j > np.asarray(t_rows)[:, None]] = -np.inf
    return s


def forward_rows(q_rows, t_rows, kv, k_pool, v_pool, page_table, P, pg,
                 k_resp, v_resp, scale):
    """O [n, Dv], LSE [n] and the probabilities p [n, P+R] for a set of rows
    that all use KV head `kv`."""
    s = scores_rows(q_rows, t_rows, kv, k_pool, page_table, P, pg, k_resp, scale)
    lse = _logsumexp_rows(s)
    p = np.exp(s - lse[:, None])
    Dv = v_resp.shape[-1]
    o = np.zeros((s.shape[0], Dv), dtype=np.float64)
    for pl, pos, valid in _page_spans(P, pg):
        vp = widen(v_pool[page_table[pl], :valid, kv, :Dv])
        o += p[:, pos:pos + valid] @ vp
    o += p[:, P:] @ widen(v_resp[:, kv, :])
    return o, lse, p


def backward_rows(q_rows, t_rows, kv, k_pool, v_pool, page_table, P, pg,
                  k_resp, v_resp, scale, d_o_rows):
    """Gradients contributed by a set of rows of one KV group.

    Returns O, LSE, dQ [n, Dk] for those rows and the rows' contributions to
    dK_resp [R, Dk] and dV_resp [R, Dv] of KV head `kv`.  The latter two are
    the complete gradients of key j only when the set holds every (t, h) with
    t >= j and h in the group.
    """
    q_rows = widen(q_rows)
    d_o_rows = widen(d_o_rows)
    o, lse, p = forward_rows(q_rows, t_rows, kv, k_pool, v_pool, page_table, P, pg,
                             k_resp, v_resp, scale)
    Dv = v_resp.shape[-1]
    Dk = k_resp.shape[-1]
    delta = (d_o_rows * o).sum(axis=1)
    dp = np.empty_like(p)
    for pl, pos, valid in _page_spans(P, pg):
        vp = widen(v_pool[page_table[pl], :valid, kv, :Dv])
        dp[:, pos:pos + valid] = d_o_rows @ vp.T
    dp[:, P:] = d_o_rows @ widen(v_resp[:, kv, :]).T
    ds = p * (dp - delta[:, None])          # masked keys have p = 0, so ds = 0
    dq = np.zeros((p.shape[0], Dk), dtype=np.float64)
    for pl, pos, valid in _page_spans(P, pg):
        kp = widen(k_pool[page_table[pl], :valid, kv, :])
        dq += ds[:, pos:pos + valid] @ kp
    dq += ds[:, P:] @ widen(k_resp[:, kv, :])
    dq *= scale
    dk_resp = scale * (ds[:, P:].T @ q_rows)
    dv_resp = p[:, P:].T @ d_o_rows
    return o, lse, dq, dk_resp, dv_resp


def replay_forward(q, k_pool, v_pool, page_table, P, pg, k_resp, v_resp, scale):
    """Full forward: O [R, Hq, Dv], LSE [R, Hq]."""
    R, Hq, _ = q.shape
    Hkv = k_resp.shape[1]
    g = Hq // Hkv
    Dv = v_resp.shape[-1]
    o = np.zeros((R, Hq, Dv))
    lse = np.zeros((R, Hq))
    t = np.arange(R)
    for h in range(Hq):
        o[:, h], lse[:, h], _ = forward_rows(q[:, h], t, h // g, k_pool, v_pool, page_table,
                                             P, pg, k_resp, v_resp, scale)
    return o, lse


def replay_backward(q, k_pool, v_pool, page_table, P, pg, k_resp, v_resp, scale, d_o):
    """Full backward: O, LSE, dQ [R,Hq,Dk], dK_resp [R,Hkv,Dk], dV_resp [R,Hkv,Dv]."""
    R, Hq, Dk = q.shape
    Hkv = k_resp.shape[1]
    g = Hq // Hkv
    Dv = v_resp.shape[-1]
    o = np.zeros((R, Hq, Dv))
    lse = np.zeros((R, Hq))
    dq = np.zeros((R, Hq, Dk))
    dk = np.zeros((R, Hkv, Dk))
    dv = np.zeros((R, Hkv, Dv))
    t = np.arange(R)
    for h in range(Hq):
        kv = h // g
        o[:, h], lse[:, h], dq[:, h], dk_h, dv_h = backward_rows(
            q[:, h], t, kv, k_pool, v_pool, page_table, P, pg, k_resp, v_resp, scale, d_o[:, h])
        dk[:, kv] += dk_h
        dv[:, kv] += dv_h
    return o, lse, dq, dk, dv


# ---------------------------------------------------------------------------
# The sharded form: Eq. qwen-local-attn per partition, then the merge.
# ---------------------------------------------------------------------------

def local_attention(q_rows, kv, k_pool, v_pool, page_table, pg, positions, scale, dv=None):
    """Eq. qwen-local-attn over the prefix positions owned by one shard:
    l_r = log sum_{j in K_r} exp(s_j),  o_r = sum exp(s_j) v_j / exp(l_r).
    An empty shard returns l_r = -inf and o_r = 0."""
    q_rows = widen(q_rows)
    positions = np.asarray(positions, dtype=np.int64)
    Dv = v_pool.shape[-1] if dv is None else dv
    n = q_rows.shape[0]
    if positions.size == 0:
        return np.zeros((n, Dv)), np.full(n, -np.inf)
    phys = np.asarray(page_table)[positions // pg]
    k = widen(k_pool[phys, positions % pg, kv, :])
    v = widen(v_pool[phys, positions % pg, kv, :Dv])
    s = scale * (q_rows @ k.T)
    l = _logsumexp_rows(s)
    o = np.exp(s - l[:, None]) @ v
    return o, l


def local_attention_response(q_rows, t_rows, kv, k_resp, v_resp, scale):
    """The causal response block as one more partition: keys j <= t."""
    q_rows = widen(q_rows)
    s = scale * (q_rows @ widen(k_resp[:, kv, :]).T)
    j = np.arange(k_resp.shape[0])[None, :]
    s[j > np.asarray(t_rows)[:, None]] = -np.inf
    l = _logsumexp_rows(s)
    o = np.exp(s - l[:, None]) @ widen(v_resp[:, kv, :])
    return o, l


def merge(o_parts, lse_parts):
    """Eq. qwen-lse-parts and Eq. qwen-global-attn over the leading axis:
    m = max_r l_r; a = sum_r e^{l_r - m}; n = sum_r e^{l_r - m} o_r;
    o = n / a; l = m + log a.  A part with l_r = -inf has weight exactly 0."""
    o_parts = np.asarray(o_parts, dtype=np.float64)
    lse_parts = np.asarray(lse_parts, dtype=np.float64)
    m = lse_parts.max(axis=0)
    m_safe = np.where(np.isfinite(m), m, 0.0)
    w = np.exp(lse_parts - m_safe)
    a = w.sum(axis=0)
    n = (w[..., None] * o_parts).sum(axis=0)
    with np.errstate(divide="ignore", invalid="ignore"):
        o = np.where(a[..., None] > 0, n / a[..., None], 0.0)
        l = m_safe + np.log(a)
    return o, l


def round_bf16(x):
    """Nearest bf16 value (8 significant bits, ties to even) of every element, as float64.
    Written out on the number itself: quantum 2^(e-7) for 2^e <= |x| < 2^(e+1) (normal range)."""
    x = np.asarray(x, dtype=np.float64)
    out = np.zeros_like(x)
    nz = (x != 0) & np.isfinite(x)
    e = np.floor(np.log2(np.abs(x[nz])))
    q = np.exp2(np.maximum(e, -126.0) - 7.0)
    out[nz] = np.rint(x[nz] / q) * q          # rint rounds halves to even
    out[~np.isfinite(x)] = x[~np.isfinite(x)]
    return out


def merge_bf16_numerator(o_parts, lse_parts):
    """The merge as the paper's production run carries it out (Sec. "Global Full-Attention Forward
    Composition", last paragraph): the numerator n = sum_r e^{l_r - m} o_r is exchanged and summed in
    bf16, the maximum, the denominator and the global LSE stay in full precision.  Reading: every
    shard's term e^{l_r - m} o_r is rounded to bf16, the terms are added in shard order and every
    running sum is rounded to bf16 again (the order of a collective's additions is not stated);
    o = n / a is then formed from the bf16 n."""
    o_parts = np.asarray(o_parts, dtype=np.float64)
    lse_parts = np.asarray(lse_parts, dtype=np.float64)
    m = lse_parts.max(axis=0)
    m_safe = np.where(np.isfinite(m), m, 0.0)
    w = np.exp(lse_parts - m_safe)
    a = w.sum(axis=0)
    n = np.zeros(o_parts.shape[1:])
    for r in range(o_parts.shape[0]):
        n = round_bf16(n + round_bf16(w[r][..., None] * o_parts[r]))
    with np.errstate(divide="ignore", invalid="ignore"):
        o = np.where(a[..., None] > 0, n / a[..., None], 0.0)
        l = m_safe + np.log(a)
    return o, l

