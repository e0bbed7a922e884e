"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every function the header declares, sizes blocks as the paper's tables say, and
rejects bad arguments before touching CUDA."""
import ctypes as C
import os
import re

import pytest

from oracle import kv_oracle as O
from paper_2604_26968_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "kvtier.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kv_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_function():
    lib = B.load()
    names = _declared()
    assert {"kv_size_bytes", "kv_epoch_score", "kv_select_victims", "kv_demote", "kv_promote"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(B.EXPORTS) == set(names)
    assert b"sm_100a" in lib.kv_version()


def _golden():
    rows = []
    for line in open(os.path.join(ROOT, "tests", "golden", "sizing.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            key, fields, _w, exp, _c = [c.strip() for c in line.split("|")]
            rows.append((key, [int(x) for x in fields.split()], int(exp)))
    return rows


@pytest.mark.parametrize("key,fields,expected", _golden())
def test_kv_size_bytes_matches_paper_tables(key, fields, expected):
    m = B.kv_model_desc(*fields)
    if key == "per_token_layer":
        got = B.kv_size_bytes(m, 1, True)
    elif key == "sequence_total":
        got = B.kv_size_bytes(m, 128000, False)
    elif key == "max_batch_mha":
        got = 8 * 30 * 10**9 // B.kv_size_bytes(m, 4096, False)
    elif key == "max_batch_arch":
        got = 30 * 10**9 // B.kv_size_bytes(m, 4096, False)
    else:
        got = B.kv_size_bytes(m, 1000, False)
    assert got == expected


def test_kv_size_bytes_agrees_with_oracle_on_a_field_sweep():
    for variant in (-1, 0, 1, 2, 3, 7):
        for hq, hkv in ((32, 32), (32, 8), (32, 1), (1, 1), (8, 32), (0, 0)):
            for lat, rope in ((0, 0), (512, 64), (3, 0)):
                for bits in (16, 8, 4, 0):
                    for n in (0, 1, 16, 4097):
                        f = (variant, 7, hq, hkv, 128, lat, rope, bits)
                        a = B.kv_size_bytes(B.kv_model_desc(*f), n, True)
                        b = O.size_bytes(O.Model(*f), n, True)
                        if variant == 7:
                            assert a < 0 and b < 0
                        else:
                            assert a == b, (f, n, a, b)
                        assert B.kv_size_bytes(B.kv_model_desc(*f), n, False) == \
                            (O.size_bytes(O.Model(*f), n, False) if variant != 7 else a)


def test_entry_bytes_of_the_five_pools():
    from paper_2604_26968_b200 import workloads as W
    expect = {1: [4096], 2: [8192], 3: [8192], 4: [73728], 5: [8192, 8192, 8192, 18432]}
    n_entries = {1: 4096, 2: 3145728, 3: 11796480, 4: 909632, 5: 18835040}
    for i, eb in expect.items():
        w = W.config(i)
        got = [B.kv_entry_bytes(B.model_desc(p), p.block_tokens) for p in w.parts]
        assert got == eb == [p.entry_bytes for p in w.parts]
        assert got == [O.entry_bytes(O.Model(p.variant, p.n_layers, p.n_q_heads, p.n_kv_heads, p.head_dim,
                                             p.d_latent, p.d_rope, p.dtype_bits), p.block_tokens)
                       for p in w.parts]
        assert w.N == n_entries[i]
    # a block whose per-head share is not a multiple of 16 bytes is refused
    assert B.kv_entry_bytes(B.kv_model_desc(B.KV_GQA, 1, 8, 2, 3, 0, 0, 16), 1) == B.KV_ERR_INVALID_ARG


def test_bad_descriptions_are_refused_without_cuda():
    lib = B.load()
    d = B.kv_pool_desc()
    dev, host = C.c_uint64(0), C.c_uint64(0)
    assert lib.kv_workspace_bytes(C.byref(d), C.byref(dev), C.byref(host)) == B.KV_ERR_INVALID_ARG
    d.n_partitions = 1
    d.part[0] = B.kv_partition_desc(B.kv_model_desc(B.KV_MLA, 4, 8, 8, 64, 0, 0, 16), 16, 0, 8, None, None, 8, None)
    assert lib.kv_workspace_bytes(C.byref(d), C.byref(dev), C.byref(host)) == B.KV_ERR_INVALID_ARG  # MLA, d_latent 0
    d.part[0] = B.kv_partition_desc(B.kv_model_desc(B.KV_GQA, 4, 8, 2, 64, 0, 0, 16), 16, 0, 8, None, None, 8, None)
    d.max_promote = 10
    assert lib.kv_workspace_bytes(C.byref(d), C.byref(dev), C.byref(host)) == B.KV_OK
    assert dev.value > 0 and host.value > 0 and dev.value % 256 == 0
    h = C.c_void_p()
    assert lib.kv_pool_create(C.byref(d), None, C.byref(h)) == B.KV_ERR_INVALID_ARG   # null pointers
    assert not h.value
    d.alpha0 = 1.0
    d.beta0 = 1.0
    for f in ("d_ema", "d_decay", "d_touch", "d_last_epoch", "d_pair", "d_state", "d_tag", "d_score",
              "d_hits", "d_misses", "d_P", "d_workspace", "h_workspace"):
        setattr(d, f, 0x1000)
    d.d_staging[0] = d.d_staging[1] = d.d_staging[2] = d.d_staging[3] = 0x1000
    d.part[0].d_slab = 0x1008                     # not 16-byte aligned
    d.part[0].h_ring = 0x1000
    d.staging_bytes = 1 << 20
    d.workspace_bytes, d.h_workspace_bytes = dev.value, host.value
    assert lib.kv_pool_create(C.byref(d), None, C.byref(h)) == B.KV_ERR_INVALID_ARG
    d.part[0].d_slab = 0x1000
    d.workspace_bytes = dev.value - 1             # workspace too small
    assert lib.kv_pool_create(C.byref(d), None, C.byref(h)) == B.KV_ERR_INVALID_ARG
    for call in (lambda: lib.kv_epoch_score(None, 0, None, None, 0, None),
                 lambda: lib.kv_select_victims(None, 1, None, None),
                 lambda: lib.kv_demote(None, None, 1, 1, None, None),
                 lambda: lib.kv_promote(None, 0, None, 1, 1, None, None)):
        assert call() == B.KV_ERR_INVALID_ARG
    assert lib.kv_status_string(B.KV_ERR_K_TOO_LARGE).decode().startswith("k exceeds")


def test_dedup_table_size_and_argument_checks_need_no_gpu():
    """The scratch table of kv_dedup_digests: a power of two, at least twice the list (so that a
    probe always ends) and at least 16; null and misaligned arguments are refused on the host."""
    for m, want in [(0, 16), (1, 16), (8, 16), (9, 32), (1000, 2048), (1024, 2048), (1025, 4096),
                    (3_145_728, 8_388_608)]:
        s = B.kv_dedup_table_slots(m)
        assert s == want and s >= 2 * m and s & (s - 1) == 0, (m, s)
    lib = B.load()
    fake = C.c_void_p(0x1000)      # aligned, never dereferenced: every call below fails its checks first
    bad = C.c_void_p(0x1004)
    args = lambda **kw: [kw.get("dig", fake), kw.get("m", 8), fake, fake, kw.get("table", fake),
                         kw.get("slots", 16), None, kw.get("status", fake), None]
    assert lib.kv_dedup_digests(*args(table=None)) == B.KV_ERR_INVALID_ARG
    assert lib.kv_dedup_digests(*args(table=bad)) == B.KV_ERR_INVALID_ARG
    assert lib.kv_dedup_digests(*args(slots=8)) == B.KV_ERR_INVALID_ARG        # fewer than 2 * m
    assert lib.kv_dedup_digests(*args(slots=24)) == B.KV_ERR_INVALID_ARG       # not a power of two
    assert lib.kv_dedup_digests(*args(status=None)) == B.KV_ERR_INVALID_ARG
    assert lib.kv_dedup_digests(*args(dig=None)) == B.KV_ERR_INVALID_ARG
    assert lib.kv_dedup_digests(*args(dig=bad)) == B.KV_ERR_INVALID_ARG
    assert lib.kv_dedup_digests(*args(m=0xFFFFFFFF, slots=1 << 34)) == B.KV_ERR_INVALID_ARG
