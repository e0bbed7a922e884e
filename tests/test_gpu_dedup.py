"""kv_hash_entries and kv_dedup_digests against the oracle (hashlib SHA-256 of the
oracle's entry images; dictionary-based reference counting): digests, stored-copy
positions and reference counts bit for bit."""
import numpy as np
import pytest

from oracle import kv_oracle as O
from paper_2604_26968_b200 import binding as B
from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _duplicate(ls, q, pairs):
    """Copies the image of entry src over entry dst (local ids of partition q) on both sides."""
    import torch
    inf = ls.ora.info(q)
    H, cb, nc = inf["H"], inf["chunk_bytes"], inf["n_chunks"]
    lb = inf["n"] // H
    o = ls.ora.part_array(q, "slab").reshape(lb, nc, H, cb)
    g = ls.gpu.pool.slabs[q][: lb * nc * H * cb].view(lb, nc, H, cb)
    for src, dst in pairs:
        o[dst // H, :, dst % H] = o[src // H, :, src % H]
        g[dst // H, :, dst % H] = g[src // H, :, src % H].clone()
    torch.cuda.synchronize()


def _gpu_digests(ls, ids, m):
    import torch
    pool = ls.gpu.pool
    d = torch.zeros((max(m, 1), 32), dtype=torch.uint8, device=pool.device)
    d_ids = None if ids is None else torch.from_numpy(np.ascontiguousarray(ids).view(np.int32)).to(pool.device)
    assert pool.kv_hash_entries(d_ids, m, d) == B.KV_OK
    pool.sync()
    assert pool.kv_device_status() == 0
    return d[:m]


def _gpu_dedup(d_digests, m):
    import torch
    dev = d_digests.device
    slots = B.kv_dedup_table_slots(m)
    assert slots >= 2 * m and slots & (slots - 1) == 0
    table = torch.empty(slots, dtype=torch.int32, device=dev)
    canon = torch.full((max(m, 1),), -1, dtype=torch.int32, device=dev)
    ref = torch.full((max(m, 1),), -1, dtype=torch.int32, device=dev)
    extra = torch.zeros(8, dtype=torch.int32, device=dev)     # [0] = n_unique, [4] = status
    assert B.kv_dedup_digests(d_digests, m, canon, ref, table, extra[0:], extra[4:]) == B.KV_OK
    torch.cuda.synchronize()
    assert int(extra[4].item()) == 0
    return canon[:m].cpu().numpy().view(np.uint32), ref[:m].cpu().numpy().view(np.uint32), int(extra[0].item())


@pytest.mark.parametrize("name,parts", [
    ("gqa 4 KB entries (pool 1)", None),
    ("mla 72 KB entries", [W.mla(3, 512, 64, 64, 40, 64, "entry")]),
    ("image sizes that leave 32, 48 and 16 bytes for the last block",
     [W.gqa(2, 4, 2, 8, 3, 50, 64, "entry"), W.mla(2, 16, 8, 1, 70, 64, "entry"), W.mla(2, 4, 4, 5, 33, 64, "entry")]),
    ("four partitions", [W.mha(2, 4, 32, 16, 30, 64, "entry"), W.gqa(3, 8, 2, 64, 16, 30, 64, "entry"),
                         W.mqa(2, 8, 128, 16, 30, 64, "entry"), W.mla(2, 512, 64, 16, 30, 64, "entry")]),
])
def test_digests_and_reference_counts_match_the_oracle(name, parts):
    from lockstep import Lockstep
    w = W.config(1) if parts is None else W.Workload("dedup", parts, 0.05, 0.02, seed=21)
    ls = Lockstep(w, payload=True, batch_bytes=256 << 10)
    ls.epoch(0)
    r = np.random.default_rng(1)
    for q, p in enumerate(w.parts):          # a fifth of every partition becomes copies of a few "system prompt" entries
        n = p.n_entries
        srcs = r.choice(n, size=4, replace=False)
        dsts = np.setdiff1d(r.choice(n, size=n // 5, replace=False), srcs)
        _duplicate(ls, q, [(int(srcs[i % 4]), int(d)) for i, d in enumerate(dsts)])
    N = w.N
    want = ls.ora.entry_digests(range(N))
    got = _gpu_digests(ls, None, N)
    assert np.array_equal(got.cpu().numpy(), want), name
    ids = r.permutation(N)[: max(N // 3, 5)].astype(np.uint32)           # a listed subset, not in id order
    got_sub = _gpu_digests(ls, ids, ids.size)
    assert np.array_equal(got_sub.cpu().numpy(), want[ids.astype(np.int64)])
    for d_dig, w_dig in ((got, want), (got_sub, want[ids.astype(np.int64)])):
        canon, ref, uniq = _gpu_dedup(d_dig, len(w_dig))
        o_canon, o_ref, o_uniq = O.dedup(w_dig)
        assert np.array_equal(canon, o_canon) and np.array_equal(ref, o_ref) and uniq == o_uniq
        assert uniq < len(w_dig)                                          # the copies were found
    ls.close()


@pytest.mark.parametrize("m,distinct", [(0, 1), (1, 1), (2, 1), (1000, 1), (4097, 4097), (200_000, 37), (300_001, 150_000)])
def test_reference_counts_on_synthetic_digests(m, distinct):
    """Many positions fighting over few digests (atomicMin under contention), and none at all."""
    import torch
    r = np.random.default_rng(m + distinct)
    base = r.integers(0, 256, (distinct, 32), dtype=np.uint8)
    base[:, :8] = base[0, :8] if distinct == 37 else base[:, :8]         # 37 digests that all probe from one slot
    dig = base[r.integers(0, distinct, m)] if m else np.zeros((0, 32), np.uint8)
    d = torch.from_numpy(np.ascontiguousarray(dig).reshape(-1)).cuda() if m else torch.zeros(32, dtype=torch.uint8).cuda()
    canon, ref, uniq = _gpu_dedup(d, m)
    o_canon, o_ref, o_uniq = O.dedup(dig)
    assert np.array_equal(canon, o_canon) and np.array_equal(ref, o_ref) and uniq == o_uniq


def test_bad_arguments_are_refused_on_the_host():
    import torch
    from paper_2604_26968_b200.harness import EpochRunner
    w = W.Workload("small", [W.gqa(1, 2, 1, 8, 1, 8, 8, "entry")], 0.1, 0.1, seed=1)
    r = EpochRunner(w, batch_bytes=4096, fill_pattern=False)
    d = torch.zeros((16, 32), dtype=torch.uint8, device=r.pool.device)
    assert r.pool.kv_hash_entries(None, 0, d) == B.KV_OK
    assert r.pool.kv_hash_entries(None, w.N + 1, d) == B.KV_ERR_INVALID_ARG        # more than there are entries
    ids = torch.tensor([0, 1, w.N, 2], dtype=torch.int32, device=r.pool.device)    # an id beyond the pool
    assert r.pool.kv_hash_entries(ids, 4, d) == B.KV_OK
    assert r.pool.kv_device_status() == B.KV_DEV_BAD_INDEX
    r.close()
    t = torch.zeros(64, dtype=torch.int32).cuda()
    assert B.kv_dedup_digests(d, 8, t, t, t[:8], t, t) == B.KV_ERR_INVALID_ARG      # table too small
    assert B.kv_dedup_digests(d, 8, t, t, t[:24], t, t) == B.KV_ERR_INVALID_ARG     # not a power of two
