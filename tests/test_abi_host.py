"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the
header declares, and rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2601_21896_b200 as pafu
from paper_2601_21896_b200 import binding as B
from paper_2601_21896_b200 import build as pbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    pbuild.build_library()
    return B.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "pafu.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pafu_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(L):
    names = declared_functions()
    assert set(names) == set(B.EXPORTS), (names, B.EXPORTS)
    for n in names:
        assert getattr(L, n) is not None
    assert L.pafu_version() >= 1000
    assert L.pafu_status_string(0) == b"ok"
    assert L.pafu_status_string(7) == b"bounded device wait ran out"


def test_struct_layouts_match_header():
    # the ctypes mirrors must have the C layout (LP64): sizes pin padding mistakes
    assert ctypes.sizeof(B.CShape) == 32
    assert ctypes.sizeof(B.CHead) == 56
    assert ctypes.sizeof(B.CPolicy) == 24
    assert ctypes.sizeof(B.CStepArgs) == 32 + 8 + 8 + 5 * 8 + 8 + 7 * 8 + 8 + 8
    assert ctypes.sizeof(B.CCache) == 4 * 4 + 3 * 8 + 6 * 8 + 8


def test_kept_counts_and_clamping(L):
    sh = pafu.Shape(12, 128, [0, 28080, 28080 + 100, 28080 + 100 + 50], None)
    pol = pafu.make_policy(1560, 4680, [14040, 200, 7], 3)
    assert pafu.pafu_kept_counts(sh, pol).tolist() == [0, 14040, 14140, 14147]
    with pytest.raises(pafu.PafuError) as e:
        pafu.pafu_kept_counts(sh, pafu.make_policy(1, 1, [5, -1, 5], 3))
    assert e.value.status == 2
    with pytest.raises(pafu.PafuError) as e:
        pafu.pafu_kept_counts(pafu.Shape(1, 64, [0, 5, 3], None), pafu.make_policy(0, 0, 1, 2))
    assert e.value.status == 1   # prefix array not monotone


def test_argument_errors_are_caught_on_the_host(L):
    vp = ctypes.c_void_p
    sh = pafu.Shape(2, 64, [0, 512], [0, 64])
    pol = pafu.make_policy(4, 64, 128, 1)
    fake = 0x10000   # never dereferenced: every call below must fail before launching
    head = B.CHead(128, 32, 1, 0, 0, fake, None, fake, None)
    assert L.pafu_score(None, fake, 4, 128, fake, None, 0, None) == 1
    assert L.pafu_score(ctypes.byref(head), None, 4, 128, fake, None, 0, None) == 1
    assert L.pafu_score(ctypes.byref(head), fake, -1, 128, fake, None, 0, None) == 1
    assert L.pafu_score(ctypes.byref(head), fake, 4, 64, fake, None, 0, None) == 1       # ldx < d_in
    assert L.pafu_score(ctypes.byref(head), fake + 2, 4, 128, fake, None, 0, None) == 5   # misaligned
    assert L.pafu_score(ctypes.byref(head), fake, 0, 128, fake, None, 0, None) == 0       # empty: no-op
    bad = B.CHead(100, 32, 1, 0, 0, fake, None, fake, None)
    assert L.pafu_score(ctypes.byref(bad), fake, 4, 128, fake, None, 0, None) == 3
    bad = B.CHead(128, 32, 1, 7, 0, fake, None, fake, None)
    assert L.pafu_score(ctypes.byref(bad), fake, 4, 128, fake, None, 0, None) == 1
    qkv = B.CHead(384, 32, 1, 0, 0, fake, None, fake, None)
    assert L.pafu_score_qkv(ctypes.byref(qkv), fake, fake, None, 4, 128, fake, None, 0, None) == 1      # V missing
    assert L.pafu_score_qkv(ctypes.byref(qkv), fake, fake, fake, 4, 64, fake, None, 0, None) == 1        # ld < d_in / 3
    assert L.pafu_score_qkv(ctypes.byref(qkv), fake, fake + 2, fake, 4, 128, fake, None, 0, None) == 5  # misaligned K
    assert L.pafu_score_qkv(ctypes.byref(head), fake, fake, fake, 4, 128, fake, None, 0, None) == 3      # 128 is not 3 x 64 k
    assert L.pafu_score_qkv(ctypes.byref(qkv), fake, fake, fake, 0, 128, fake, None, 0, None) == 0      # empty: no-op
    assert L.pafu_select(None, ctypes.byref(sh.c), pol, fake, None, 0, None) == 1
    assert L.pafu_select(fake, ctypes.byref(sh.c), None, fake, None, 0, None) == 1
    assert L.pafu_select(fake, ctypes.byref(sh.c), pafu.make_policy(-1, 0, 5, 1), fake, None, 0, None) == 2
    assert L.pafu_select(fake, None, pol, fake, None, 0, None) == 1
    assert L.pafu_compact(fake, fake, None, fake, ctypes.byref(sh.c), pol, fake, fake + 4096, None, None) == 1  # aliasing
    assert L.pafu_compact(fake, fake + 4096, None, None, ctypes.byref(sh.c), pol, fake + 8192, fake + 12288, None, None) == 1
    assert L.pafu_compact(fake, fake + 4096, fake, fake, ctypes.byref(sh.c), pol, fake + 8192, fake + 12288, None, None) == 1
    cu_B = np.array([0, 128], dtype=np.int64)
    sh3 = pafu.Shape(2, 96, [0, 512], [0, 64])
    assert L.pafu_chunk_attn(fake, fake, fake, cu_B.ctypes.data, fake, fake, ctypes.byref(sh3.c), 0.0, fake, None, None, 0, None) == 3
    assert L.pafu_chunk_attn(fake, fake, fake, cu_B.ctypes.data, fake, None, ctypes.byref(sh.c), 0.0, fake, None, None, 0, None) == 1
    assert L.pafu_chunk_attn(fake, fake, fake, cu_B.ctypes.data, fake, fake, ctypes.byref(sh.c), -1.0, fake, None, None, 0, None) == 1
    assert L.pafu_chunk_attn(fake, fake, fake, None, fake, fake, ctypes.byref(sh.c), 0.0, fake, None, None, 0, None) == 1
    too_many = pafu.Shape(2, 64, list(range(0, 35)), list(range(0, 35)))
    assert L.pafu_select(fake, ctypes.byref(too_many.c), pafu.make_policy(0, 0, 1, 34), fake, None, 0, None) == 3
    assert L.pafu_step(None, None) == 1
    assert L.pafu_workspace_status(None, None) == 1
    assert L.pafu_workspace_bytes(None, None, None) == 0
    assert L.pafu_workspace_bytes(ctypes.byref(sh.c), pol, None) >= 256
    assert L.pafu_workspace_bytes(ctypes.byref(sh.c), pol, None) % 256 == 0


def test_newer_entry_points_reject_bad_arguments_on_host(L):
    fake = 0x7f0000000000
    sh = pafu.Shape(2, 128, [0, 512], [0, 64])
    sh64 = pafu.Shape(2, 64, [0, 512], [0, 64])
    pol = pafu.make_policy(4, 64, 128, 1)
    cu_B = np.array([0, 128], dtype=np.int64)
    # attention through indices: d_head 128 only, idx required, retained count cannot exceed the cache
    call = lambda shape, idx, cb: L.pafu_chunk_attn_indexed(fake, fake, fake, idx, cb.ctypes.data, fake, fake,
                                                            ctypes.byref(shape.c), 0.0, fake, None, fake, 1 << 30, None)
    assert call(sh64, fake, cu_B) == 3
    assert call(sh, None, cu_B) == 1
    assert call(sh, fake, np.array([0, 513], dtype=np.int64)) == 1
    assert call(sh, fake + 4, cu_B) == 5
    assert L.pafu_step_indexed(None, None) == 1
    # all-layer compaction: pointer arrays, layer count
    arr = (ctypes.c_void_p * 2)(fake, fake + 4096)
    out = (ctypes.c_void_p * 2)(fake + 8192, fake + 12288)
    cl = lambda K, n, Kc: L.pafu_compact_layers(K, arr, n, None, fake, ctypes.byref(sh.c), pol, Kc, out, None, None)
    assert cl(arr, -1, out) == 1
    assert cl(arr, 65, out) == 3
    assert cl(None, 2, out) == 1
    assert cl(arr, 2, arr) == 1                                     # in place
    assert cl((ctypes.c_void_p * 2)(fake, None), 2, out) == 1       # a missing layer
    assert cl(arr, 0, out) == 0                                     # no layers: no-op
    # teacher salience target
    sse = lambda Lt, N, D, LB, scale, s, ws, nb: L.pafu_sse(fake, fake, None, Lt, N, D, LB, scale, s, None, None, None, ws, nb, None)
    need = L.pafu_sse_workspace_bytes(1000, 2, 128, 256)
    assert need > 0 and need % 256 == 0
    assert L.pafu_sse_workspace_bytes(1000, 2, 64, 256) == 0 and L.pafu_sse_workspace_bytes(0, 2, 128, 256) == 0
    assert sse(1000, 2, 64, 256, 0.0, fake, fake, need) == 3
    assert sse(0, 2, 128, 256, 0.0, fake, fake, need) == 1
    assert sse(1000, 2, 128, 0, 0.0, fake, fake, need) == 1
    assert sse(1000, 2, 128, 256, -1.0, fake, fake, need) == 1
    assert sse(1000, 2, 128, 256, 0.0, None, fake, need) == 1
    assert sse(1000, 2, 128, 256, 0.0, fake, fake + 16, need) == 5
    assert sse(1000, 2, 128, 256, 0.0, fake, fake, need - 1) == 4


def test_overlap_and_host_step_checks_run_before_anything_is_enqueued(L):
    """Outputs that overlap inputs are rejected by range, not only by equal pointers; and the
    host-buffer step validates the whole head before its first copy (every call below returns an
    argument error with fake pointers that must never be touched)."""
    fake = 0x7f0000000000
    sh = pafu.Shape(2, 128, [0, 512], [0, 64])                 # 512 cache rows of 512 bytes, 128 kept
    pol = pafu.make_policy(4, 64, 128, 1)
    K, V = fake, fake + (1 << 20)
    inside_K = fake + 512 * 512 - 1024                          # starts inside K's last rows
    ok_Kc, ok_Vc = fake + (2 << 20), fake + (3 << 20)
    cp = lambda Kc, Vc, SL=None, SLc=None: L.pafu_compact(K, V, SL, fake + (4 << 20), ctypes.byref(sh.c), pol, Kc, Vc, SLc, None)
    assert cp(inside_K, ok_Vc) == 1                             # Kc overlaps K
    assert cp(ok_Kc, V + 4096) == 1                             # Vc overlaps V
    assert cp(ok_Kc, ok_Kc + 1024) == 1                         # the two outputs overlap each other
    assert cp(ok_Kc, ok_Vc, fake + (5 << 20), fake + (5 << 20) + 256) == 1    # SLc inside SL
    # host-buffer step: bad head sizes / enums / scale are caught before any copy
    head = lambda d_in, d_hid, act: B.CHead(d_in, d_hid, 1, act, 0, fake, None, fake, None)
    pol1 = ctypes.cast(pol, ctypes.POINTER(B.CPolicy))
    def args(h, scale=0.0):
        a = B.CStepArgs(sh.c, ctypes.pointer(h), pol1, fake, fake, fake, fake, fake, scale, fake, fake, None, None, None,
                        fake, None, None, 0)
        a._keep = h
        return a
    arena = 0x7f1000000000
    big = 1 << 40
    assert L.pafu_step_host(ctypes.byref(args(head(256, 17, 0))), arena, big, None) == 3     # d_hidden % 16
    assert L.pafu_step_host(ctypes.byref(args(head(256, 32, 9))), arena, big, None) == 1     # activation enum
    assert L.pafu_step_host(ctypes.byref(args(head(192, 32, 0))), arena, big, None) == 1     # d_in != heads * d_head
    assert L.pafu_step_host(ctypes.byref(args(head(256, 32, 0), -1.0)), arena, big, None) == 1
    assert L.pafu_step_host(ctypes.byref(args(head(256, 32, 0))), arena + 8, big, None) == 5  # arena alignment
    assert L.pafu_step_host(ctypes.byref(args(head(256, 32, 0))), arena, 1024, None) == 4     # arena too small
    assert L.pafu_workspace_counters(None, None, None) == 1


def test_cache_update_rejects_bad_arguments_on_host(L):
    """Every refusal of pafu_cache_update comes before anything is enqueued and leaves the
    host counters as they were (fake device addresses: nothing may be touched)."""
    fake = 0x7f0000000000
    n_layers, N, D, cap, chunk = 2, 2, 64, 1024, 256
    dm, MB = N * D, 1 << 20
    def make(cur=0, T=0, capacity=cap, share=False, sl_same=False):
        ptrs = lambda base: (ctypes.c_void_p * n_layers)(*[base + l * MB for l in range(n_layers)])
        arrs = [ptrs(fake + 16 * MB), ptrs(fake + (16 if share else 32) * MB), ptrs(fake + 48 * MB), ptrs(fake + 64 * MB)]
        c = B.CCache()
        c.n_layers, c.n_heads, c.d_head, c.cur, c.capacity, c.n_sink, c.T = n_layers, N, D, cur, capacity, 16, T
        c.K[0], c.K[1] = ctypes.cast(arrs[0], ctypes.c_void_p), ctypes.cast(arrs[1], ctypes.c_void_p)
        c.V[0], c.V[1] = ctypes.cast(arrs[2], ctypes.c_void_p), ctypes.cast(arrs[3], ctypes.c_void_p)
        c.SL[0], c.SL[1] = fake + 96 * MB, fake + (96 if sl_same else 97) * MB
        c.idx = fake + 98 * MB
        return c, arrs
    head = B.CHead(3 * dm, 64, 12, 1, 0, fake + 100 * MB, None, fake + 101 * MB, None)
    new = (ctypes.c_void_p * n_layers)(fake + 110 * MB, fake + 111 * MB)
    def call(c, ch=chunk, hd=head, kn=new, ws=fake + 120 * MB, nb=1 << 20):
        pr = ctypes.c_int32(7)
        rc = L.pafu_cache_update(ctypes.byref(c), ctypes.byref(hd) if hd is not None else None, fake, fake, fake, kn, new, ch,
                                 ctypes.byref(pr), ws, nb, None)
        return rc, pr.value
    c, keep = make(T=300)
    assert call(c, ch=cap + 1) == (8, 0) and (c.T, c.cur) == (300, 0)          # chunk longer than the cache
    assert call(c, ch=-1)[0] == 1
    assert call(c, ch=0) == (0, 0) and c.T == 300                               # nothing to append: no-op
    assert call(make(cur=2)[0])[0] == 1
    assert call(make(T=cap + 1)[0])[0] == 1
    assert call(make(share=True)[0])[0] == 1                                    # the two buffer sets share storage
    assert call(make(sl_same=True)[0])[0] == 1
    assert call(c, hd=None)[0] == 1
    assert call(c, hd=B.CHead(2 * dm, 64, 12, 1, 0, fake, None, fake, None))[0] == 1   # head does not read [q, k, v]
    assert call(c, kn=(ctypes.c_void_p * n_layers)(fake + 110 * MB, None))[0] == 1
    assert call(c, kn=(ctypes.c_void_p * n_layers)(fake + 110 * MB, fake + 111 * MB + 2))[0] == 5
    assert call(c, kn=(ctypes.c_void_p * n_layers)(fake + 16 * MB, fake + 111 * MB))[0] == 1   # new rows inside a cache buffer
    assert call(c, ws=None)[0] == 1
    assert call(c, ws=fake + 120 * MB + 64)[0] == 5
    assert call(c, nb=16)[0] == 4
    c65, _ = make(); c65.n_layers = 65
    assert call(c65)[0] == 3
    assert (c.T, c.cur) == (300, 0)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU path"):
        B.lib()
