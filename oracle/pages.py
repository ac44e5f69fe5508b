"""Integer page and shard arithmetic of the resident prefix (oracle side).

Test infrastructure only; independent of the CUDA library's host planner.

Notation follows the paper: P prefix positions, page size pg, Np logical pages,
C (here S) context-parallel shards.  Positions and masks stay in the original
sequence coordinates (Sec. "From Logical Shards to Physical Pages").
"""
import numpy as np

CONTIGUOUS = 0   # shard s = one contiguous run of logical pages
CYCLIC = 1       # Eq. qwen-page-owner: owner(p) = p mod C
ZIGZAG = 2       # Eq. glm-tr-zigzag-pages: chunks r and 2C-1-r of 2C chunks


def num_pages(P, pg):
    """Eq. qwen-page-count generalised: Np = ceil(P / pg)."""
    if P < 0 or pg <= 0:
        raise ValueError("bad P or page size")
    return (P + pg - 1) // pg


def last_page_valid(P, pg):
    """Valid tokens in the last logical page (pg when P divides, 0 when P = 0)."""
    if P == 0:
        return 0
    r = P % pg
    return pg if r == 0 else r


def _even_chunks(n, parts):
    """Cut range(n) into `parts` contiguous chunks; the first n % parts chunks
    hold one page more.  Returns the parts+1 chunk boundaries."""
    base, rem = divmod(n, parts)
    bounds = [0]
    for c in range(parts):
        bounds.append(bounds[-1] + base + (1 if c < rem else 0))
    return bounds


def shard_page_lists(Np, S, policy):
    """For every shard, its logical pages in local storage order."""
    if S <= 0:
        raise ValueError("need at least one shard")
    if policy == CONTIGUOUS:
        b = _even_chunks(Np, S)
        return [np.arange(b[s], b[s + 1], dtype=np.int64) for s in range(S)]
    if policy == CYCLIC:
        return [np.arange(s, Np, S, dtype=np.int64) for s in range(S)]
    if policy == ZIGZAG:
        b = _even_chunks(Np, 2 * S)
        out = []
        for r in range(S):
            lo = np.arange(b[r], b[r + 1], dtype=np.int64)
            m = 2 * S - 1 - r
            hi = np.arange(b[m], b[m + 1], dtype=np.int64)
            out.append(np.concatenate([lo, hi]))
        return out
    raise ValueError("unknown shard policy")


def shard_of_page(Np, S, policy):
    """owner[p] for every logical page p."""
    owner = np.full(Np, -1, dtype=np.int32)
    for s, pages in enumerate(shard_page_lists(Np, S, policy)):
        owner[pages] = s
    assert (owner >= 0).all()
    return owner


def shard_tokens(P, pg, S, policy):
    """Valid prefix tokens held by every shard (last logical page may be short)."""
    Np = num_pages(P, pg)
    out = np.zeros(S, dtype=np.int64)
    for s, pages in enumerate(shard_page_lists(Np, S, policy)):
        n = len(pages) * pg
        if len(pages) and pages.max() == Np - 1:
            n -= pg - last_page_valid(P, pg)
        out[s] = n
    return out


def shard_positions(P, pg, S, policy):
    """Global prefix positions of every shard, in local storage order."""
    Np = num_pages(P, pg)
    out = []
    for pages in shard_page_lists(Np, S, policy):
        pos = (pages[:, None] * pg + np.arange(pg, dtype=np.int64)[None, :]).reshape(-1)
        out.append(pos[pos < P])
    return out


def check_page_table(page_table, Np, num_phys_pages):
    """A valid table maps the Np logical pages one-to-one into the pool."""
    t = np.asarray(page_table)
    if t.shape != (Np,):
        return False
    if Np == 0:
        return True
    if t.min() < 0 or t.max() >= num_phys_pages:
        return False
    return len(np.unique(t)) == Np


def kv_payload_bytes(layers, pages, pg, kv_heads, head_dim, elem_bytes=2, tensors=2):
    """Eq. qwen-kv-bytes: raw K and V payload of `pages` pages over `layers` layers."""
    return layers * pages * tensors * pg * kv_heads * head_dim * elem_bytes
