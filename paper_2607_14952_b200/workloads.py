"""Seeded synthetic workloads shaped like the paper's replay runs.

This module only draws random inputs; it holds none of the method's arithmetic
and is the one piece the tests hand to both the CUDA library and the CPU oracle.

The paper's long-context runs use synthetic random tokens (Sec. "Four-Block
Response Replay": 24 query heads, 4 KV heads, head dim 256, bf16 KV pages,
2,048-token response blocks; GLM route: 64 heads over one 576-wide latent), so
i.i.d. N(0,1) bf16 Q/K/V/dO at those shapes stand in for them.
"""
from dataclasses import dataclass, replace
import numpy as np
import torch


@dataclass(frozen=True)
class ReplayConfig:
    name: str
    P: int            # prefix positions
    R: int            # response tokens
    Hq: int
    Hkv: int
    Dk: int
    Dv: int
    page_size: int
    num_shards: int
    G: int            # group members replayed serially against one prefix
    cycles: int = 1   # optimizer cycles reusing the resident prefix
    needles: int = 0  # prefix keys set to 4x a query vector
    v_aliases_k: bool = False   # MLA: V is the first Dv channels of the K page
    seed: int = 0

    @property
    def scale(self):
        return float(1.0 / np.sqrt(np.float64(self.Dk)))

    @property
    def num_pages(self):
        return (self.P + self.page_size - 1) // self.page_size


CONFIGS = {
    "tiny": ReplayConfig("tiny", 4096, 256, 4, 1, 128, 128, 64, 4, 1, seed=1001),
    "p128k": ReplayConfig("p128k", 131072, 2048, 24, 4, 256, 256, 256, 8, 2, seed=2001),
    "p2m": ReplayConfig("p2m", 2097152, 4096, 24, 4, 256, 256, 256, 8, 8, needles=16, seed=3001),
    "p4m": ReplayConfig("p4m", 4456448, 2048, 24, 4, 256, 256, 512, 8, 8, cycles=8, seed=4001),
    "mla1m": ReplayConfig("mla1m", 1048576, 1024, 64, 1, 576, 512, 64, 32, 2,
                          v_aliases_k=True, seed=5001),
}


def scaled(cfg, **kw):
    """A smaller or altered copy of a config (tests use this for ragged cases)."""
    return replace(cfg, **kw)


def _splitmix64(state):
    state = (state + 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
    z = state
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
    return state, z ^ (z >> 31)


def page_permutation(num_logical, num_phys, seed):
    """Logical -> physical page table: Fisher-Yates over range(num_phys) driven by
    splitmix64(seed), truncated to the first num_logical entries."""
    perm = list(range(num_phys))
    st = seed & 0xFFFFFFFFFFFFFFFF
    for i in range(num_phys - 1, 0, -1):
        st, r = _splitmix64(st)
        j = r % (i + 1)
        perm[i], perm[j] = perm[j], perm[i]
    return np.asarray(perm[:num_logical], dtype=np.int32)


def _randn_bf16(shape, seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    step = 1 << 28
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        out[lo:hi] = torch.randn(hi - lo, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    return out.view(*shape)


def member_seed(cfg, member, cycle=0):
    return cfg.seed + 10 * (member + 1) + 1000 * cycle


def make_member(cfg, member, device="cpu", cycle=0):
    """Q [R,Hq,Dk], K_resp [R,Hkv,Dk], V_resp [R,Hkv,Dv], dO [R,Hq,Dv] of one group member."""
    s = member_seed(cfg, member, cycle)
    q = _randn_bf16((cfg.R, cfg.Hq, cfg.Dk), s + 0, device)
    k = _randn_bf16((cfg.R, cfg.Hkv, cfg.Dk), s + 1, device)
    v = _randn_bf16((cfg.R, cfg.Hkv, cfg.Dv), s + 2, device)
    d_o = _randn_bf16((cfg.R, cfg.Hq, cfg.Dv), s + 3, device)
    return q, k, v, d_o


def needle_plan(cfg):
    """For needle n: (prefix position, member, response row, query head)."""
    rng = np.random.default_rng(cfg.seed + 3)
    pos = rng.choice(cfg.P, size=cfg.needles, replace=False) if cfg.needles else np.zeros(0, int)
    plan = []
    for n in range(cfg.needles):
        plan.append((int(pos[n]), n % cfg.G, int(rng.integers(cfg.R)), int(rng.integers(cfg.Hq))))
    return plan


def make_prefix(cfg, device="cpu", extra_phys_pages=0, permute=True):
    """Physical page pools and the logical->physical page table.

    Returns k_pool [Nphys,pg,Hkv,Dk], v_pool [Nphys,pg,Hkv,Dv] (a view of k_pool's
    first Dv channels when cfg.v_aliases_k) and page_table int32 [Np].
    Needle keys are 4x the raw query vector of their (member, row, head).
    """
    Np = cfg.num_pages
    nphys = Np + extra_phys_pages
    k_pool = _randn_bf16((nphys, cfg.page_size, cfg.Hkv, cfg.Dk), cfg.seed + 0, device)
    if cfg.v_aliases_k:
        v_pool = k_pool[..., :cfg.Dv]
    else:
        v_pool = _randn_bf16((nphys, cfg.page_size, cfg.Hkv, cfg.Dv), cfg.seed + 1, device)
    if permute:
        table = page_permutation(Np, nphys, cfg.seed + 2)
    else:
        table = np.arange(Np, dtype=np.int32)
    g = cfg.Hq // cfg.Hkv
    q_cache = {}
    for pos, member, t, h in needle_plan(cfg):
        if member not in q_cache:
            q_cache[member] = _randn_bf16((cfg.R, cfg.Hq, cfg.Dk), member_seed(cfg, member), device)
        vec = (4.0 * q_cache[member][t, h].float()).to(torch.bfloat16)
        k_pool[int(table[pos // cfg.page_size]), pos % cfg.page_size, h // g] = vec
    return k_pool, v_pool, table


def make_index_inputs(cfg, num_index_heads, member=0, device="cpu", index_dim=128, num_phys_pages=None):
    """Indexer side of the sparse (DSA) replay (Eq. dsa-index): indexer-key pages
    [num_phys_pages, page_size, index_dim] bf16 (seed base+4; they follow the latent's page table),
    the member's indexer queries [R, H_I, index_dim] bf16 and head weights [R, H_I] fp32."""
    nphys = cfg.num_pages if num_phys_pages is None else num_phys_pages
    ki_pool = _randn_bf16((nphys, cfg.page_size, index_dim), cfg.seed + 4, device)
    s = member_seed(cfg, member)
    q_index = _randn_bf16((cfg.R, num_index_heads, index_dim), s + 4, device)
    g = torch.Generator(device=device)
    g.manual_seed(s + 5)
    w_index = torch.randn((cfg.R, num_index_heads), generator=g, device=device, dtype=torch.float32)
    return ki_pool, q_index, w_index


def bf16_bits(t):
    """torch bf16 tensor -> numpy uint16 bit patterns (host copy)."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)
