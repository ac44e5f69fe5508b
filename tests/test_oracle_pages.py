"""Pins for the oracle's integer page/shard arithmetic: the paper's worked examples
(tests/golden/paper_page_examples.json) and partition invariants."""
import json
import os

import numpy as np
import pytest

from oracle import pages as op

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_page_examples.json")))


def test_paper_block_cyclic_example():
    g = GOLD["qwen_block_cyclic"]
    assert g["prompt_tokens"] + g["response_tokens"] == g["total_positions"]
    Np = op.num_pages(g["prompt_tokens"], g["page_size"])
    assert Np == g["pages"]
    lists = op.shard_page_lists(Np, g["cp"], op.CYCLIC)
    assert all(len(l) == g["pages_per_rank"] for l in lists)
    owner = op.shard_of_page(Np, g["cp"], op.CYCLIC)
    assert (owner == np.arange(Np) % g["cp"]).all()
    b = op.kv_payload_bytes(g["layers"], g["pages_per_rank"], g["page_size"], g["kv_heads"],
                            g["head_dim"], g["bytes_per_elem"])
    assert b == g["kv_bytes_per_rank"]


def test_paper_zigzag_example():
    g = GOLD["glm_zigzag"]
    Np = op.num_pages(g["prompt_tokens"], g["page_size"])
    assert Np == g["pages"]
    lists = op.shard_page_lists(Np, g["cp"], op.ZIGZAG)
    for r, key in ((0, "rank0"), (31, "rank31")):
        (a0, a1), (b0, b1) = g[key]
        want = np.concatenate([np.arange(a0, a1 + 1), np.arange(b0, b1 + 1)])
        assert (lists[r] == want).all()
    assert all(len(l) == g["pages_per_rank"] for l in lists)
    assert (op.shard_tokens(g["prompt_tokens"], g["page_size"], g["cp"], op.ZIGZAG) == g["tokens_per_rank"]).all()
    # rank r owns chunk r and its mirror 2C-1-r
    r = 5
    c = g["pages_per_chunk"]
    assert lists[r][0] == c * r and lists[r][c] == c * (2 * g["cp"] - 1 - r)


def test_paper_page_payloads():
    g = GOLD["glm_page_payload"]
    assert op.kv_payload_bytes(1, g["pages"], g["page_size"], 1, g["mla_width"], 2, tensors=1) == g["mla_bytes"]
    assert op.kv_payload_bytes(1, g["pages"], g["page_size"], 1, g["dsa_width"], 2, tensors=1) == g["dsa_bytes"]
    assert g["mla_bytes"] == 72 * 2**20 and g["dsa_bytes"] == 16 * 2**20


@pytest.mark.parametrize("policy", [op.CONTIGUOUS, op.CYCLIC, op.ZIGZAG])
@pytest.mark.parametrize("P,pg,S", [(4096, 64, 4), (1000, 64, 3), (63, 64, 4), (0, 64, 2), (130, 64, 8), (64 * 7, 64, 2)])
def test_partition_invariants(policy, P, pg, S):
    Np = op.num_pages(P, pg)
    lists = op.shard_page_lists(Np, S, policy)
    assert len(lists) == S
    allp = np.concatenate(lists) if Np else np.zeros(0, int)
    assert sorted(allp.tolist()) == list(range(Np))          # every page owned exactly once
    for l in lists:                                           # ascending within contiguous/cyclic
        if policy != op.ZIGZAG:
            assert (np.diff(l) > 0).all()
    toks = op.shard_tokens(P, pg, S, policy)
    assert toks.sum() == P
    pos = op.shard_positions(P, pg, S, policy)
    assert [len(x) for x in pos] == toks.tolist()
    assert sorted(np.concatenate(pos).tolist()) == list(range(P))
    owner = op.shard_of_page(Np, S, policy)
    for s, l in enumerate(lists):
        assert (owner[l] == s).all()


def test_contiguous_uneven_split_rule():
    # first Np mod S shards hold one page more
    lists = op.shard_page_lists(10, 4, op.CONTIGUOUS)
    assert [len(l) for l in lists] == [3, 3, 2, 2]
    assert lists[1].tolist() == [3, 4, 5]


def test_last_page_valid_and_table_check():
    assert op.last_page_valid(4096, 64) == 64
    assert op.last_page_valid(4097, 64) == 1
    assert op.last_page_valid(0, 64) == 0
    assert op.check_page_table(np.array([2, 0, 1]), 3, 3)
    assert op.check_page_table(np.array([5, 0, 1]), 3, 6)
    assert not op.check_page_table(np.array([2, 2, 1]), 3, 3)      # duplicate
    assert not op.check_page_table(np.array([3, 0, 1]), 3, 3)      # out of range
    assert not op.check_page_table(np.array([-1, 0, 1]), 3, 3)
    assert not op.check_page_table(np.array([0, 1]), 3, 3)         # wrong length
