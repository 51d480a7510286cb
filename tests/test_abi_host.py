"""Host-side checks of the C ABI (no GPU): the library loads, exports what include/kata.h
declares, and rejects bad arguments with the documented status codes before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2607_17419_b200 import binding as kb
from paper_2607_17419_b200 import build as kbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    kbuild.build()
    return kb.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "kata.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kata_[a-z_]+)\s*\(", text)))


def test_exports_match_header(L):
    names = declared_functions()
    assert set(names) == set(kb.EXPORTS)
    for n in names:
        assert hasattr(L, n), n


def test_version_and_status_strings(L):
    assert kb.kata_version() == 100
    seen = {kb.status_string(s) for s in range(0, -8, -1)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert kb.status_string(-99) == "unknown status"


def test_opts_struct_layout():
    assert ctypes.sizeof(kb.KataOpts) == 96
    assert kb.KataOpts.workspace.offset == 32 and kb.KataOpts.stream.offset == 72
    assert kb.KataOpts.s_init.offset == 80 and kb.KataOpts.z_init.offset == 88


def call(L, fn, q=256, k=512, v=768, out=1024, B=1, H=1, T=64, d_k=64, d_v=64, C=64, opts=None):
    opts = opts if opts is not None else kb.make_opts(kb.KATA_BF16)
    return getattr(L, fn)(q, k, v, out, B, H, T, d_k, d_v, C, ctypes.byref(opts))


@pytest.mark.parametrize("fn", ["kata_fwd_quadratic", "kata_fwd_chunked", "kata_chunk_state_scan"])
def test_invalid_arguments(L, fn):
    INV, SHAPE, ALIGN, WS = -1, -2, -3, -4
    assert getattr(L, fn)(256, 512, 768, 1024, 1, 1, 64, 64, 64, 64, None) == INV
    bad = kb.make_opts(kb.KATA_BF16)
    bad.struct_size = 12
    assert call(L, fn, opts=bad) == INV
    assert call(L, fn, q=None) == INV
    assert call(L, fn, out=None) == INV
    assert call(L, fn, B=0) == INV
    assert call(L, fn, T=0) == INV
    assert call(L, fn, opts=kb.make_opts(7)) == INV
    assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, feature_order=3)) == INV
    assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, scan_group=-1)) == INV
    assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, s_pre=4096)) == INV       # z_pre missing
    assert call(L, fn, d_k=48) == SHAPE
    assert call(L, fn, d_v=128) == SHAPE
    assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, impl=kb.KATA_IMPL_TENSOR)) == SHAPE
    assert call(L, fn, q=260) == ALIGN
    assert call(L, fn, out=1032) == ALIGN
    if fn != "kata_fwd_quadratic":
        assert call(L, fn, C=32) == SHAPE
        assert call(L, fn, C=0) == INV
    if fn == "kata_chunk_state_scan":
        assert call(L, fn, T=640) == WS                                        # needs a workspace
        o = kb.make_opts(kb.KATA_F32, workspace=4096 + 8, workspace_bytes=1 << 40)
        assert call(L, fn, T=640, opts=o) == ALIGN
        o = kb.make_opts(kb.KATA_F32, s_pre=4096, z_pre=8192, scan_group=4)
        assert call(L, fn, T=640, opts=o) == INV
    elif fn == "kata_fwd_chunked":
        # final-state export: sequential form and the PSD feature only
        assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, s_pre=4096, z_pre=8192, inter_chunk=kb.KATA_SCAN)) == INV
        assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, s_pre=4096, z_pre=8192, feature_order=1)) == SHAPE
        assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, s_pre=4096)) == INV
        assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, s_pre=4096, z_pre=8192)) == WS          # fp32 path: one internal state per head
        # initial state: the same rules
        assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, s_init=4096)) == INV
        assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, z_init=4096)) == INV
        assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, s_init=4096, z_init=8192, inter_chunk=kb.KATA_SCAN)) == INV
        assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, s_init=4096, z_init=8192, feature_order=1)) == SHAPE
        assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, s_init=4096, z_init=8192)) == WS
        assert call(L, fn, opts=kb.make_opts(kb.KATA_BF16, s_init=4096 + 4, z_init=8192)) == ALIGN
        # the tensor-core path takes the state without a workspace (unless it is advanced in place: a copy of the
        # normaliser state); narrower rows with a state go through the fp32 path
        o = kb.make_opts(kb.KATA_BF16, s_init=4096, z_init=8192)
        assert kb.kata_workspace_bytes(kb.KATA_FN_CHUNKED, 1, 1, 64, 64, 64, 64, o) == 0
        o = kb.make_opts(kb.KATA_BF16, s_init=4096, z_init=8192, feature_groups=2)
        assert kb.kata_workspace_bytes(kb.KATA_FN_CHUNKED, 1, 1, 64, 64, 64, 64, o) == 0
        o = kb.make_opts(kb.KATA_BF16, s_init=4096, z_init=8192, s_pre=4096, z_pre=8192, feature_groups=2)
        assert kb.kata_workspace_bytes(kb.KATA_FN_CHUNKED, 1, 1, 64, 64, 64, 64, o) == 2 * 32 * 32 * 4
        o = kb.make_opts(kb.KATA_BF16, s_init=4096, z_init=8192)
        assert kb.kata_workspace_bytes(kb.KATA_FN_CHUNKED, 1, 1, 64, 32, 32, 64, o) > 0
    else:
        assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, s_pre=4096, z_pre=8192)) == INV
        assert call(L, fn, opts=kb.make_opts(kb.KATA_F32, s_init=4096, z_init=8192)) == INV


def test_scan_workspace_and_plan(L):
    o = kb.make_opts(kb.KATA_BF16)
    # tensor-core quadratic path: one bf16 scale per key (the values are used as they are)
    assert kb.kata_workspace_bytes(kb.KATA_FN_QUADRATIC, 4, 16, 4096, 64, 64, 64, o) == 4 * 16 * 4096 * 2
    o32 = kb.make_opts(kb.KATA_F32)
    assert kb.kata_workspace_bytes(kb.KATA_FN_QUADRATIC, 4, 16, 4096, 64, 64, 64, o32) == 0
    # sequential walk of the feature-split kernel: tile counters and the ticket, the scaled values and key scales of
    # the pre-pass, nine shares of 17 KB per head and tile of 128 tokens
    al = lambda x: (x + 255) // 256 * 256
    BH, T, nt = 8 * 16, 4096, 32
    assert kb.kata_workspace_bytes(kb.KATA_FN_CHUNKED, 8, 16, 4096, 64, 64, 64, o) == \
        al((BH * nt + 1) * 4) + al(BH * T * 64 * 2) + al(BH * T * 2) + al(BH * 9 * nt * (128 * 128 + 128 * 8))
    assert kb.kata_scan_plan(kb.KATA_FN_CHUNKED, 8, 16, 4096, 64, 64, 64, o)[0] == 1
    o = kb.make_opts(kb.KATA_BF16, inter_chunk=kb.KATA_SCAN, scan_group=16, impl=kb.KATA_IMPL_SIMT)
    ng, g, rounds = kb.kata_scan_plan(kb.KATA_FN_CHUNKED, 1, 16, 8192, 64, 64, 64, o)
    assert (ng, g, rounds) == (8, 16, 3)
    assert kb.kata_workspace_bytes(kb.KATA_FN_CHUNKED, 1, 16, 8192, 64, 64, 64, o) > 0
    # per-chunk pipeline: T=2048, C=64 -> 32 chunks; the exclusive prefix needs the inclusive scan of
    # the first 31 chunk states: ceil(log2 31) = 5 rounds
    o = kb.make_opts(kb.KATA_F32, impl=kb.KATA_IMPL_SIMT)
    assert kb.kata_scan_plan(kb.KATA_FN_CHUNK_STATE_SCAN, 1, 2, 2048, 16, 16, 64, o) == (32, 1, 5)
    assert kb.kata_scan_plan(kb.KATA_FN_CHUNK_STATE_SCAN, 1, 2, 4160, 16, 16, 64, o) == (65, 1, 6)
    # host-I/O variant adds the staging area
    a = kb.kata_workspace_bytes(kb.KATA_FN_CHUNK_STATE_SCAN, 1, 2, 2048, 16, 16, 64, o)
    b = kb.kata_workspace_bytes(kb.KATA_FN_CHUNK_STATE_SCAN | kb.KATA_FN_HOST_IO, 1, 2, 2048, 16, 16, 64, o)
    assert b >= a + 4 * 2 * 2048 * 16 * 4
    assert kb.kata_workspace_bytes(kb.KATA_FN_CHUNKED, 1, 1, 64, 48, 64, 64, o) == 0      # invalid -> 0


def test_inter_chunk_auto_and_tensor_groups(L):
    """inter_chunk = AUTO: the scan form only where few heads leave the GPU idle on a long sequence, never with a
    state hand-off, never on the fp32 kernels; the tensor-core scan form's own grouping fills whole waves."""
    auto = kb.make_opts(kb.KATA_BF16, inter_chunk=kb.KATA_INTER_AUTO)
    plan = lambda B, H, T, o: kb.kata_scan_plan(kb.KATA_FN_CHUNKED, B, H, T, 64, 64, 64, o)
    assert plan(8, 16, 4096, auto)[0] == 1                    # 1024 CTAs: sequential
    assert plan(1, 16, 131072, auto)[0] == 1                  # 128 CTAs already fill 148 SMs
    ng, g, rounds = plan(1, 1, 131072, auto)                  # 8 CTAs per group: 18 groups make one wave of 144
    assert (ng, g) == (18, 114) and rounds == 5
    assert plan(1, 4, 131072, auto)[0] > 1
    assert plan(1, 1, 256, auto)[0] == 1                      # two tiles: nothing to gain
    auto32 = kb.make_opts(kb.KATA_F32, inter_chunk=kb.KATA_INTER_AUTO)
    assert plan(1, 1, 131072, auto32)[0] == 1
    hand = kb.make_opts(kb.KATA_BF16, inter_chunk=kb.KATA_INTER_AUTO, s_pre=4096, z_pre=8192)
    assert plan(1, 1, 131072, hand)[0] == 1
    bad = kb.make_opts(kb.KATA_BF16, inter_chunk=3)
    with pytest.raises(kb.KataError):
        plan(1, 1, 1024, bad)
    # explicit scan form on the tensor cores: groups of whole 128-token tiles, the last pass in whole waves
    scan = kb.make_opts(kb.KATA_BF16, inter_chunk=kb.KATA_SCAN)
    ng, g, _ = plan(1, 16, 131072, scan)
    assert (ng, g) == (2, 1024)
    ng, g, _ = plan(1, 4, 131072, scan)
    assert g % 2 == 0 and (ng - 1) * g < 2048 <= ng * g


def test_host_entry_piece_plan(L):
    """The host-buffer entry works piece by piece only on long sequences of the sequential chunked form on the
    tensor-core path: at least four pieces of at least 8192 tokens, at most sixteen, whole 128-token tiles."""
    o = kb.make_opts(kb.KATA_BF16)
    plan = lambda fn, B, H, T, opts=o, d=64: kb.kata_host_plan(fn, B, H, T, d, d, 64, opts)
    assert plan(kb.KATA_FN_CHUNKED, 1, 16, 131072) == (16, 8192)
    assert plan(kb.KATA_FN_CHUNKED, 1, 2, 32768) == (4, 8192)
    pieces, tokens = plan(kb.KATA_FN_CHUNKED, 1, 1, 70001)
    assert tokens % 128 == 0 and (pieces - 1) * tokens < 70001 <= pieces * tokens and pieces == 8
    assert plan(kb.KATA_FN_CHUNKED, 1, 16, 32767) == (1, 32767)                  # too short
    assert plan(kb.KATA_FN_QUADRATIC, 1, 16, 65536) == (1, 65536)                # needs every key
    assert plan(kb.KATA_FN_CHUNK_STATE_SCAN, 1, 16, 131072) == (1, 131072)
    assert plan(kb.KATA_FN_CHUNKED, 1, 16, 131072, kb.make_opts(kb.KATA_BF16, inter_chunk=kb.KATA_SCAN)) == (1, 131072)
    assert plan(kb.KATA_FN_CHUNKED, 1, 16, 131072, kb.make_opts(kb.KATA_F32)) == (1, 131072)      # fp32 kernels
    assert plan(kb.KATA_FN_CHUNKED, 1, 16, 131072, kb.make_opts(kb.KATA_BF16, impl=kb.KATA_IMPL_SIMT)) == (1, 131072)
    assert plan(kb.KATA_FN_CHUNKED, 1, 16, 131072, kb.make_opts(kb.KATA_BF16, feature_order=1)) == (1, 131072)
    assert plan(kb.KATA_FN_CHUNKED, 1, 16, 131072, o, d=32) == (1, 131072)       # padded rows
    assert plan(kb.KATA_FN_CHUNKED, 1, 16, 131072, kb.make_opts(kb.KATA_BF16, feature_groups=2)) == (16, 8192)
    assert plan(kb.KATA_FN_CHUNKED, 1, 16, 131072, kb.make_opts(kb.KATA_BF16, s_pre=4096, z_pre=8192)) == (1, 131072)
    # the pieces fit the workspace the host entry asks for anyway
    with pytest.raises(kb.KataError):
        plan(kb.KATA_FN_CHUNKED, 0, 16, 131072)


def test_no_oracle_in_product_path():
    """The package must not import or reference the oracle."""
    pkg = os.path.join(ROOT, "paper_2607_17419_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+\S*oracle", text, flags=re.M), f
                assert "kata_oracle" not in text and "oracle/" not in text, f


def test_decode_step_argument_checks(L):
    INV, SHAPE, ALIGN, WS = -1, -2, -3, -4
    def dec(q=4096, k=4096, v=4096, out=4096, S=4096, Z=4096, B=2, H=2, dk=64, dv=64, opts=None):
        o = opts if opts is not None else kb.make_opts(kb.KATA_F32, workspace=4096, workspace_bytes=1 << 30)
        return L.kata_decode_step(q, k, v, out, S, Z, B, H, dk, dv, ctypes.byref(o))

    assert dec(q=0) == INV and dec(S=0) == INV and dec(Z=0) == INV and dec(B=0) == INV
    assert dec(dk=48) == SHAPE and dec(dv=8) == SHAPE
    assert dec(S=4100) == ALIGN and dec(out=4104) == ALIGN
    assert dec(opts=kb.make_opts(kb.KATA_F32)) == WS                                     # needs a workspace
    assert dec(opts=kb.make_opts(kb.KATA_F32, workspace=4096, workspace_bytes=64)) == WS
    assert dec(opts=kb.make_opts(kb.KATA_F32, workspace=4096 + 8, workspace_bytes=1 << 30)) == ALIGN
    assert dec(opts=kb.make_opts(kb.KATA_F32, workspace=4096, workspace_bytes=1 << 30, s_pre=4096, z_pre=8192)) == INV
    # workspace: one partial numerator row and denominator per 256 feature rows of every head, rounded up to 256 B
    up = lambda n: (n + 255) // 256 * 256
    o = kb.make_opts(kb.KATA_BF16)
    assert kb.kata_workspace_bytes(kb.KATA_FN_DECODE_STEP, 2, 3, 1, 64, 64, 0, o) == up(2 * 3 * 16 * 65 * 4)
    o = kb.make_opts(kb.KATA_BF16, state_layout=kb.KATA_LAYOUT_PACKED)
    assert kb.kata_workspace_bytes(kb.KATA_FN_DECODE_STEP, 2, 3, 1, 64, 32, 0, o) == up(2 * 3 * 9 * 33 * 4)
    o = kb.make_opts(kb.KATA_F32, feature_order=1)
    assert kb.kata_workspace_bytes(kb.KATA_FN_DECODE_STEP, 1, 1, 1, 16, 16, 0, o) == 256   # 17 floats, rounded up
    assert kb.decode_n_psi(64) == 4096 and kb.decode_n_psi(64, 2, kb.KATA_LAYOUT_PACKED) == 2080 and kb.decode_n_psi(64, 1) == 64


def test_backward_argument_checks(L):
    INV, SHAPE, ALIGN, WS = -1, -2, -3, -4
    def bwd(q=4096, k=4096, v=4096, dout=4096, dq=4096, dk=4096, dv=4096, B=2, H=2, T=100, d_k=64, d_v=64, opts=None):
        o = opts if opts is not None else kb.make_opts(kb.KATA_F32, workspace=4096, workspace_bytes=1 << 30)
        return L.kata_bwd_quadratic(q, k, v, dout, dq, dk, dv, B, H, T, d_k, d_v, ctypes.byref(o))

    assert bwd(q=0) == INV and bwd(dout=0) == INV and bwd(dv=0) == INV and bwd(T=0) == INV
    assert bwd(d_k=48) == SHAPE and bwd(d_v=8) == SHAPE
    assert bwd(dq=4100) == ALIGN
    assert bwd(opts=kb.make_opts(kb.KATA_F32)) == WS
    assert bwd(opts=kb.make_opts(kb.KATA_F32, workspace=4096, workspace_bytes=1 << 30, impl=kb.KATA_IMPL_TENSOR)) == SHAPE
    assert bwd(opts=kb.make_opts(kb.KATA_F32, workspace=4096, workspace_bytes=1 << 30, feature_groups=3)) == INV
    assert bwd(opts=kb.make_opts(kb.KATA_F32, workspace=4096, workspace_bytes=1 << 30, s_pre=4096, z_pre=8192)) == INV
    up = lambda n: (n + 255) // 256 * 256
    rows = 2 * 3 * 100
    # fp32 kernels: two floats per row; tensor-core kernels (bf16, d = 64): k' (bf16), r and the two row scalars (fp32)
    o = kb.make_opts(kb.KATA_F32)
    assert kb.kata_workspace_bytes(kb.KATA_FN_BWD_QUADRATIC, 2, 3, 100, 64, 64, 0, o) == up(rows * 2 * 4)
    o = kb.make_opts(kb.KATA_BF16)
    assert kb.kata_workspace_bytes(kb.KATA_FN_BWD_QUADRATIC, 2, 3, 100, 64, 64, 0, o) == up(rows * 128) + up(rows * 4) + up(rows * 8)
    o = kb.make_opts(kb.KATA_BF16, feature_groups=2)          # blockwise map at d = 64: tensor-core kernels too
    assert kb.kata_workspace_bytes(kb.KATA_FN_BWD_QUADRATIC, 2, 3, 100, 64, 64, 0, o) == up(rows * 128) + up(rows * 4) + up(rows * 8)
    assert kb.kata_workspace_bytes(kb.KATA_FN_BWD_QUADRATIC, 2, 3, 100, 32, 32, 0, o) == up(rows * 2 * 4)     # narrower: fp32 kernels
    # narrower bf16 rows: seven padded tensors in front of the tensor-core scratch
    o = kb.make_opts(kb.KATA_BF16)
    assert kb.kata_workspace_bytes(kb.KATA_FN_BWD_QUADRATIC, 2, 3, 100, 32, 16, 0, o) == \
        7 * up(rows * 128) + up(rows * 128) + up(rows * 4) + up(rows * 8)


def test_more_heads_than_a_grid_axis(L):
    """Beyond 65535 heads the forward device entries work in slabs: the scratch is the largest slab's, the plan a full
    slab's; state pointers, the backward, the decode step and the host-buffer entry keep the limit."""
    SHAPE, WS = -2, -4
    o = kb.make_opts(kb.KATA_F32)
    for fn in (kb.KATA_FN_CHUNKED, kb.KATA_FN_CHUNK_STATE_SCAN):
        ws = lambda B, H, opts=o: kb.kata_workspace_bytes(fn, B, H, 300, 16, 16, 64, opts)
        assert ws(65537, 1) == max(ws(1, 65535), ws(1, 2)) and ws(70000, 2) == max(ws(1, 65535), ws(1, 140000 % 65535))
        assert kb.kata_scan_plan(fn, 65537, 1, 300, 16, 16, 64, o) == kb.kata_scan_plan(fn, 1, 65535, 300, 16, 16, 64, o)
    assert kb.kata_workspace_bytes(kb.KATA_FN_QUADRATIC, 300, 300, 5, 16, 16, 64, o) == 0
    # a slab's scratch is checked before anything is launched
    need = kb.kata_workspace_bytes(kb.KATA_FN_CHUNK_STATE_SCAN, 65537, 1, 300, 16, 16, 64, o)
    small = kb.make_opts(kb.KATA_F32, workspace=4096, workspace_bytes=need - 256)
    assert call(L, "kata_chunk_state_scan", B=65537, T=300, d_k=16, d_v=16, opts=small) == WS
    states = kb.make_opts(kb.KATA_F32, workspace=4096, workspace_bytes=1 << 40, s_init=4096, z_init=8192)
    assert call(L, "kata_fwd_chunked", B=65537, T=300, d_k=16, d_v=16, opts=states) == SHAPE
    ob = kb.make_opts(kb.KATA_F32, workspace=4096, workspace_bytes=1 << 40)
    assert L.kata_bwd_quadratic(4096, 4096, 4096, 4096, 4096, 4096, 4096, 65537, 1, 8, 16, 16, ctypes.byref(ob)) == SHAPE
    assert L.kata_decode_step(4096, 4096, 4096, 4096, 4096, 4096, 65537, 1, 16, 16, ctypes.byref(ob)) == SHAPE
