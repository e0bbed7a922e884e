"""Pins for the oracle's content hashing and deduplication.

The paper indexes blocks by the SHA-256 hash of their content and counts
references instead of storing a block twice (content-addressable deduplication
section).  SHA-256 itself is fixed by FIPS 180-4: the oracle's hashing step is
checked against the standard's published example digests.  What "content of a
block" means here (the entry image: K chunk then V chunk) is checked against a
slab written by hand from the layout definition; the reference counting against
a quadratic brute force.
"""
import os

import numpy as np
import pytest

from oracle import kv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "sha256.txt")


def _vectors():
    out = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        spec, digest = line.rsplit(" ", 1)
        if spec == "empty":
            msg = b""
        elif spec.startswith("ascii:"):
            msg = spec[6:].encode()
        else:
            _, ch, n = spec.split(":")
            msg = ch.encode() * int(n)
        out.append((spec[:24], msg, digest))
    return out


@pytest.mark.parametrize("name,msg,digest", _vectors())
def test_hash_step_reproduces_the_published_digests(name, msg, digest):
    got = O.sha256_bytes(np.frombuffer(msg, dtype=np.uint8))
    assert got.tobytes().hex() == digest


def test_entry_image_is_k_chunk_then_v_chunk_of_that_head():
    # GQA, 2 layers, 3 KV heads, 4 tokens of dim 8 in 16 bits: chunk = 64 bytes
    part = dict(model=O.model(variant=O.GQA, n_layers=2, n_q_heads=6, n_kv_heads=3, head_dim=8),
                block_tokens=4, blocks_per_layer=5, ring_slots=8)
    p = O.OraclePool([part], n_tags=64, payload=True)
    L, NB, H, cb = 2, 5, 3, 4 * 8 * 2
    slab = p.part_array(0, "slab")
    r = np.random.default_rng(3)
    slab[:] = r.integers(0, 256, slab.size, dtype=np.uint8)
    view = slab.reshape(L, NB, 2, H, cb)           # [layer][block][K,V][head][token*dim bytes]
    for layer, block, head in [(0, 0, 0), (1, 4, 2), (0, 3, 1)]:
        i = (layer * NB + block) * H + head
        img = p.entry_image(i)
        assert img.size == 2 * cb
        assert np.array_equal(img[:cb], view[layer, block, 0, head])     # K
        assert np.array_equal(img[cb:], view[layer, block, 1, head])     # V
    d = p.entry_digests([7, 8])
    assert d.shape == (2, 32)
    assert np.array_equal(d[0], O.sha256_bytes(p.entry_image(7)))
    assert not np.array_equal(d[0], d[1])


def test_mla_image_is_the_single_chunk():
    part = dict(model=O.model(variant=O.MLA, n_layers=2, n_q_heads=4, n_kv_heads=4, head_dim=8,
                              d_latent=24, d_rope=8), block_tokens=4, blocks_per_layer=3, ring_slots=8)
    p = O.OraclePool([part], n_tags=64, payload=True)
    slab = p.part_array(0, "slab")
    slab[:] = np.arange(slab.size, dtype=np.uint64).astype(np.uint8)
    eb = 4 * 32 * 2
    for i in range(6):
        assert np.array_equal(p.entry_image(i), slab[i * eb:(i + 1) * eb])


def test_dedup_against_quadratic_brute_force():
    r = np.random.default_rng(11)
    for n, distinct in [(0, 1), (1, 1), (40, 7), (200, 200), (300, 3)]:
        base = r.integers(0, 256, (distinct, 32), dtype=np.uint8)
        digests = base[r.integers(0, distinct, n)] if n else np.zeros((0, 32), np.uint8)
        canon, ref, uniq = O.dedup(digests)
        want_canon = [min(i for i in range(n) if np.array_equal(digests[i], digests[j])) for j in range(n)]
        assert canon.tolist() == want_canon
        assert ref.tolist() == [want_canon.count(i) if want_canon[i] == i else 0 for i in range(n)]
        assert uniq == len(set(want_canon))
        assert int(ref.sum()) == n


def test_identical_blocks_share_a_digest_and_a_flipped_bit_separates_them():
    part = dict(model=O.model(variant=O.GQA, n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=8),
                block_tokens=4, blocks_per_layer=4, ring_slots=8)
    p = O.OraclePool([part], n_tags=64, payload=True)
    slab = p.part_array(0, "slab")
    slab[:] = np.random.default_rng(5).integers(0, 256, slab.size, dtype=np.uint8)
    view = slab.reshape(1, 4, 2, 2, 64)
    view[0, 2, :, 1] = view[0, 0, :, 0]            # entry (block 2, head 1) := entry (block 0, head 0)
    a, b = 0, 2 * 2 + 1
    d = p.entry_digests([a, b])
    assert np.array_equal(d[0], d[1])
    view[0, 2, 1, 1, 63] ^= 1                      # last byte of the V chunk
    assert not np.array_equal(p.entry_digests([b])[0], d[0])
    canon, ref, uniq = O.dedup(p.entry_digests(range(8)))
    assert uniq == 8
