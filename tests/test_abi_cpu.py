"""CPU-side checks of the C ABI: the library builds, loads and exports what include/astro.h declares,
and host-only argument validation and ring metadata behave as documented (no kernel is launched)."""
import ctypes as C
import os
import re

import pytest

from paper_2603_17051_b200 import binding as A

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "astro.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(astro_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = A.lib()
    names = declared_functions()
    assert len(names) >= 13
    for n in names:
        assert hasattr(L, n), n
    assert sorted(A.EXPORTED) == [n for n in names if n in A.EXPORTED]
    assert set(names) == set(A.EXPORTED)


def test_status_strings():
    seen = set()
    for code in range(9):
        s = A.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 9
    assert A.status_string(99) == "unknown status"


def test_storage_and_workspace_bytes():
    assert A.astro_kvcache_storage_bytes(1, 12, 128, 1560, 3, 18) == 12 * 21 * 1560 * 128 * 2
    assert A.astro_kvcache_storage_bytes(4, 12, 128, 1560, 3, 12) == 4 * 12 * 15 * 1560 * 128 * 2
    assert A.astro_kvcache_storage_bytes(1, 12, 96, 1560, 3, 18) == 0      # head_dim must be 64 or 128
    assert A.astro_kvcache_storage_bytes(1, 12, 128, 1560, 3, 0) == 0       # window needs a slot
    assert A.astro_chunk_attn_bwd_workspace_bytes(2, 12, 4680, 128) == 2 * 12 * 4680 * 4 + (-(2 * 12 * 4680 * 4)) % 256
    assert A.astro_chunk_attn_bwd_workspace_bytes(2, 12, 4680, 100) == 0


def _raw_create(desc, k=0x10000, v=0x20000, nbytes=1 << 40):
    out = C.c_void_p()
    st = A.lib().astro_kvcache_create(C.byref(desc) if desc is not None else None, C.c_void_p(k), C.c_void_p(v),
                                      nbytes, C.byref(out))
    return st, out


def test_create_validation_and_ring_metadata_without_a_device():
    L = A.lib()
    d = A.KVCacheDesc(1, 2, 64, 16, 1, 4)
    assert _raw_create(None)[0] == 1
    assert _raw_create(d, k=0)[0] == 1
    assert _raw_create(A.KVCacheDesc(1, 2, 80, 16, 1, 4))[0] == 2
    assert _raw_create(d, k=0x10008)[0] == 3
    assert _raw_create(d, nbytes=100)[0] == 4
    st, h = _raw_create(d)
    assert st == 0
    a, b, c = C.c_int(-1), C.c_int(-1), C.c_int64(-1)
    assert L.astro_kvcache_query(h, C.byref(a), C.byref(b), C.byref(c)) == 0
    assert (a.value, b.value, c.value) == (0, 0, 0)
    # evict on an empty window underflows; negative counts are shape errors; zero is fine
    assert L.astro_kvcache_evict(h, 1, None) == 5
    assert L.astro_kvcache_evict(h, -1, None) == 2
    assert L.astro_kvcache_evict(h, 0, None) == 0
    # capacity is checked before anything touches the device: S+L = 5 frames
    assert L.astro_kvcache_append(h, C.c_void_p(0x30000), C.c_void_p(0x40000), 6, None) == 4
    assert L.astro_kvcache_append(h, None, C.c_void_p(0x40000), 1, None) == 1
    assert L.astro_kvcache_append(h, C.c_void_p(0x30004), C.c_void_p(0x40000), 1, None) == 3
    assert L.astro_kvcache_append(h, C.c_void_p(0x30000), C.c_void_p(0x40000), 0, None) == 0
    assert L.astro_kvcache_reset(h) == 0
    assert L.astro_kvcache_destroy(h) == 0
    assert L.astro_kvcache_destroy(None) == 1


def test_attention_argument_validation_happens_before_any_launch():
    L = A.lib()
    p = C.c_void_p(0x10000)
    lse = C.c_void_p(0x50000)
    # no key at all
    assert L.astro_chunk_attn_fwd(None, p, None, None, 1, 2, 64, 48, 0, 0.125, p, lse, None) == 2
    # unsupported head_dim, negative scale, null q
    assert L.astro_chunk_attn_fwd(None, p, p, p, 1, 2, 96, 48, 48, 0.125, p, lse, None) == 2
    assert L.astro_chunk_attn_fwd(None, p, p, p, 1, 2, 64, 48, 48, -1.0, p, lse, None) == 2
    assert L.astro_chunk_attn_fwd(None, None, p, p, 1, 2, 64, 48, 48, 0.125, p, lse, None) == 1
    assert L.astro_chunk_attn_fwd(None, C.c_void_p(0x10002), p, p, 1, 2, 64, 48, 48, 0.125, p, lse, None) == 3
    # cache with other head count / batch
    st, h = _raw_create(A.KVCacheDesc(2, 2, 64, 16, 0, 4))
    assert st == 0
    assert L.astro_chunk_attn_fwd(h, p, p, p, 3, 2, 64, 48, 48, 0.125, p, lse, None) == 2
    assert L.astro_chunk_attn_fwd(h, p, p, p, 2, 4, 64, 48, 48, 0.125, p, lse, None) == 2
    # backward: workspace too small, null dO
    assert L.astro_chunk_attn_bwd(None, p, p, p, p, lse, p, 1, 2, 64, 48, 48, 0.125, p, p, p, p, 16, None) == 4
    assert L.astro_chunk_attn_bwd(None, p, p, p, p, lse, None, 1, 2, 64, 48, 48, 0.125, p, p, p, p, 4096, None) == 1
    L.astro_kvcache_destroy(h)


def test_product_never_reaches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2603_17051_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle|#include.*oracle|oracle[./]", text, flags=re.M), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2603_17051_b200" not in text and "ctypes" not in text, f


def test_state_record_round_trip_and_validation():
    L = A.lib()
    st, h = _raw_create(A.KVCacheDesc(1, 2, 64, 16, 2, 4))
    assert st == 0
    rec = A.KVCacheState()
    assert L.astro_kvcache_get_state(h, C.byref(rec)) == 0
    assert (rec.sink_held, rec.window_head, rec.window_held, rec.frames_seen) == (0, 0, 0, 0)
    good = A.KVCacheState(2, 3, 4, 17)
    assert L.astro_kvcache_set_state(h, C.byref(good)) == 0
    assert L.astro_kvcache_get_state(h, C.byref(rec)) == 0
    assert (rec.sink_held, rec.window_head, rec.window_held, rec.frames_seen) == (2, 3, 4, 17)
    a, b, c = C.c_int(), C.c_int(), C.c_int64()
    L.astro_kvcache_query(h, C.byref(a), C.byref(b), C.byref(c))
    assert (a.value, b.value, c.value) == (2, 4, 17)
    assert L.astro_kvcache_evict(h, 3, None) == 0                      # ring index advances modulo L
    L.astro_kvcache_get_state(h, C.byref(rec))
    assert (rec.window_head, rec.window_held) == (2, 1)
    for bad in (A.KVCacheState(3, 0, 0, 3), A.KVCacheState(2, 4, 1, 9), A.KVCacheState(2, 0, 5, 9),
                A.KVCacheState(1, 0, 2, 9), A.KVCacheState(2, 0, 2, 3), A.KVCacheState(-1, 0, 0, 0)):
        assert L.astro_kvcache_set_state(h, C.byref(bad)) == 2
    assert L.astro_kvcache_set_state(h, None) == 1
    L.astro_kvcache_destroy(h)


def test_header_compiles_as_c_and_links(tmp_path):
    """include/astro.h is a C header: build a C99 program against it and the shared library, run it."""
    import shutil
    import subprocess
    from paper_2603_17051_b200 import build as B
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    A.lib()
    exe = str(tmp_path / "c_abi_check")
    cmd = [gcc, "-std=c99", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(ROOT, "include"),
           os.path.join(ROOT, "tests", "c_abi_check.c"), "-o", exe, "-L", B.LIB_DIR, "-lastro",
           "-Wl,-rpath," + B.LIB_DIR]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    run = subprocess.run([exe], capture_output=True, text=True)
    assert run.returncode == 0 and "c abi ok" in run.stdout, run.stdout + run.stderr


def test_key_segments_cover_exactly_the_held_slots_in_every_ring_state():
    """Host logic the kernels rely on: for every (sink, ring head, window count) state the cache segments are
    disjoint, at most two, merged where adjacent, and cover exactly the tokens of the held slots."""
    L = A.lib()
    for S, Lw, T in ((0, 1, 3), (0, 4, 5), (2, 3, 7), (3, 5, 2)):
        st, h = _raw_create(A.KVCacheDesc(1, 1, 64, T, S, Lw))
        assert st == 0
        n, a, b, c = C.c_int(), (C.c_int * 3)(), (C.c_int * 3)(), (C.c_int * 3)()
        states = [(sink, 0, 0) for sink in range(S + 1)] + [(S, head, held) for head in range(Lw) for held in range(1, Lw + 1)]
        for sink, head, held in states:
            rec = A.KVCacheState(sink, head, held, sink + held + 10)
            assert L.astro_kvcache_set_state(h, C.byref(rec)) == 0
            for n_kc in (0, 9):
                assert L.astro_kvcache_key_segments(h, n_kc, C.byref(n), a, b, c) == 0
                segs = [(a[i], b[i], c[i]) for i in range(n.value)]
                cache_segs = [s for s in segs if s[2] == 0]
                chunk_segs = [s for s in segs if s[2] == 1]
                assert chunk_segs == ([(0, n_kc, 1)] if n_kc else []) and (not chunk_segs or segs[-1] == chunk_segs[0])
                assert len(cache_segs) <= 2
                slots = list(range(sink)) + [S + (head + i) % Lw for i in range(held)]
                expect = sorted(t for sl in slots for t in range(sl * T, (sl + 1) * T))
                got = sorted(t for f, cnt, _ in cache_segs for t in range(f, f + cnt))
                assert got == expect, (S, Lw, sink, head, held)
                assert len(set(got)) == len(got)
                cache_segs.sort()
                for x, y in zip(cache_segs, cache_segs[1:]):
                    assert x[0] + x[1] < y[0]                      # adjacent ranges were merged
        L.astro_kvcache_destroy(h)
    # no cache at all: only the chunk
    assert A.astro_kvcache_key_segments(None, 5) == [(0, 5, 1)]


def test_two_threads_share_one_handle_for_validation_and_inspection():
    """Attention calls take the cache as const: several host threads may issue them on one handle (the G candidates
    of a group decoding against one shared prefix).  Here two threads hammer argument validation and the
    key-segment inspection of one handle at the same time; every call must return the same answers as alone.
    (What the calls do after validation needs a device and is covered by the GPU tests.)"""
    import threading
    L = A.lib()
    d = A.KVCacheDesc(1, 2, 64, 16, 1, 4)
    st, h = _raw_create(d)
    assert st == 0
    vp = C.c_void_p
    results = [[], []]

    def worker(slot):
        n = C.c_int(); a, b, c = (C.c_int * 3)(), (C.c_int * 3)(), (C.c_int * 3)()
        for _ in range(2000):
            # misaligned q: rejected before anything is launched or any lazily built state is touched
            r1 = L.astro_chunk_attn_fwd(h, vp(0x1008), vp(0x2000), vp(0x3000), 1, 2, 64, 8, 8, 0.1, vp(0x4000), None, None)
            # a cache of other heads: shape error
            r2 = L.astro_chunk_attn_fwd(h, vp(0x1000), vp(0x2000), vp(0x3000), 1, 3, 64, 8, 8, 0.1, vp(0x4000), None, None)
            r3 = L.astro_kvcache_key_segments(h, 5, C.byref(n), a, b, c)
            results[slot].append((r1, r2, r3, n.value, a[0], b[0], c[0]))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads: t.start()
    for t in threads: t.join()
    expect = (3, 2, 0, 1, 0, 5, 1)                       # ALIGN, SHAPE, OK and one chunk segment of 5 tokens
    assert all(r == expect for res in results for r in res)
    assert L.astro_kvcache_destroy(h) == 0


def test_static_backward_rejects_misaligned_outputs_before_any_launch():
    """A misaligned dK is an ASTRO_ERR_ALIGN up front (no device is needed to get the answer: nothing ran)."""
    L = A.lib()
    vp = C.c_void_p
    st = L.astro_chunk_attn_bwd_static(None, vp(0x1000), vp(0x2000), vp(0x3000), vp(0x4000), vp(0x5000), vp(0x6000),
                                       1, 2, 64, 8, 8, 0.1, vp(0x7000), vp(0x8008), vp(0x9000), None)
    assert st == 3
