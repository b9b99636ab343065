"""CPU checks of the C-ABI boundary: the shared library loads, exports every function that
include/vsa.h declares, and rejects bad arguments on the host with the documented codes.
No kernel is launched here (every call below fails validation before touching the device)."""
import ctypes as C
import os
import re

import pytest

from paper_2602_13804_b200 import binding as B
from paper_2602_13804_b200 import build as vsa_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "vsa.h")


@pytest.fixture(scope="module")
def lib():
    vsa_build.build()
    return B.lib()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vsa_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert {"vsa_build_page_summaries", "vsa_route_pages", "vsa_sparse_decode", "vsa_dense_decode_fallback",
            "vsa_decode_step", "vsa_decode_step_host", "vsa_workspace_bytes", "vsa_strerror"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in vsa.h but not exported by libvsa.so"


def test_struct_layouts_match_the_header():
    assert C.sizeof(B.vsa_diag_t) == 32
    assert C.sizeof(B.vsa_shape_t) == 6 * 4 + 4 * 8
    assert B.vsa_shape_t.num_pool_pages.offset == 24


def test_strerror_covers_all_codes(lib):
    texts = {c: B.vsa_strerror(c) for c in (0, -1, -2, -3, -4, -5, -6, -99)}
    assert texts[0] == "ok" and "unknown" in texts[-99]
    assert len(set(texts.values())) == len(texts)


def test_workspace_sizes(lib):
    s = B.make_shape(8, 32, 8, 2048, 65536)
    route = B.vsa_workspace_bytes(s, 32, 256, B.VSA_WS_ROUTE)
    assert route == 8 * 32 * 2048 * 4          # one fp32 score per (unit, logical page)
    assert B.vsa_workspace_bytes(s, 32, 256, B.VSA_WS_SPARSE) == 0
    dense = B.vsa_workspace_bytes(s, 32, 256, B.VSA_WS_DENSE)
    assert dense > 0
    assert B.vsa_workspace_bytes(s, 32, 256, B.VSA_WS_STEP) >= route + dense
    bad = B.make_shape(8, 32, 8, 2048, 65536, head_dim=96)
    assert B.vsa_workspace_bytes(bad, 32, 256, B.VSA_WS_STEP) == 0
    assert B.vsa_workspace_bytes(s, 32, 256, 77) == 0


FAKE = 0x10000   # an aligned non-NULL address that is never dereferenced: validation fails first
ODD = 0x10008    # not 16-byte aligned


def _route(lib, shape, q=FAKE, summ=FAKE, bt=FAKE, sl=FAKE, P=32, routed=FAKE, ws=FAKE, ws_bytes=1 << 40):
    return lib.vsa_route_pages(C.byref(shape) if shape is not None else None, q, summ, bt, sl, P, routed, None,
                               ws, ws_bytes, None)


def test_route_argument_validation(lib):
    ok = B.make_shape(2, 8, 2, 64, 256)
    assert _route(lib, None) == -1
    assert _route(lib, ok, q=None) == -1
    assert _route(lib, ok, routed=None) == -1
    assert _route(lib, ok, ws=None) == -1
    assert _route(lib, ok, P=0) == -1
    assert _route(lib, ok, P=129) == -2
    assert _route(lib, B.make_shape(2, 8, 2, 64, 256, head_dim=96)) == -2
    assert _route(lib, B.make_shape(2, 8, 2, 64, 256, page_size=64)) == -2
    assert _route(lib, B.make_shape(2, 6, 2, 64, 256)) == -2          # group of 3
    assert _route(lib, B.make_shape(2, 7, 2, 64, 256)) == -1          # heads do not divide
    assert _route(lib, B.make_shape(0, 8, 2, 64, 256)) == -1
    assert _route(lib, B.make_shape(2, 8, 2, 40000, 256)) == -2       # block-table row too wide
    assert _route(lib, ok, ws_bytes=16) == -3
    assert _route(lib, ok, q=ODD) == -4
    assert _route(lib, B.make_shape(2, 8, 2, 64, 256, kv_token_stride=132)) == -4
    assert _route(lib, B.make_shape(2, 8, 2, 64, 256, kv_token_stride=64)) == -1


def _sparse(lib, shape, P=4, K_c=16, eps=1.0, tau=0.0, out=FAKE, diag=FAKE, fl=FAKE, fc=FAKE, q=FAKE):
    return lib.vsa_sparse_decode(C.byref(shape), q, FAKE, FAKE, FAKE, FAKE, FAKE, P, K_c, eps, tau, out, diag, fl,
                                 fc, None, 0, None)


def test_sparse_argument_validation(lib):
    ok = B.make_shape(2, 8, 2, 64, 256)
    assert _sparse(lib, ok, eps=0.0) == -1
    assert _sparse(lib, ok, eps=-1.0) == -1
    assert _sparse(lib, ok, eps=float("inf")) == -1
    assert _sparse(lib, ok, eps=float("nan")) == -1
    assert _sparse(lib, ok, tau=float("nan")) == -1
    assert _sparse(lib, ok, K_c=0) == -1
    assert _sparse(lib, ok, K_c=4 * 16 + 1) == -2
    assert _sparse(lib, ok, out=None) == -1
    assert _sparse(lib, ok, diag=None) == -1
    assert _sparse(lib, ok, fc=None) == -1
    assert _sparse(lib, ok, q=ODD) == -4


def test_entropic_argument_validation(lib):
    ok = B.make_shape(2, 8, 2, 64, 256)
    s = C.byref(ok)

    def call(P=32, K_c=16, iters=4, solve=FAKE, eps=1.0):
        return lib.vsa_sparse_decode_entropic(s, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, P, K_c, eps, 0.0, iters, FAKE, FAKE,
                                              solve, FAKE, FAKE, None)

    assert call(K_c=257) == -2             # more candidates than the on-chip tile holds
    assert call(iters=-1) == -1 and call(iters=65) == -1
    assert call(solve=None) == -1
    assert call(eps=0.0) == -1
    assert call(P=4, K_c=65) == -2
    fw = lib.vsa_sparse_decode_frank_wolfe
    assert fw(s, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 32, 257, 1.0, 0.0, 2, FAKE, FAKE, FAKE, FAKE, FAKE, None) == -2
    assert fw(s, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 32, 16, 1.0, 0.0, 65, FAKE, FAKE, FAKE, FAKE, FAKE, None) == -1
    assert fw(s, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 32, 16, 1.0, 0.0, 2, FAKE, FAKE, None, FAKE, FAKE, None) == -1
    fws = lib.vsa_decode_step_frank_wolfe
    assert fws(s, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 32, 16, 1.0, 0.0, 2, FAKE, FAKE, None, FAKE, FAKE, FAKE, FAKE,
               1 << 40, None) == -1
    step = lib.vsa_decode_step_entropic
    assert step(s, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 32, 257, 1.0, 0.0, 2, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE,
                1 << 40, None) == -2
    assert step(s, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 32, 16, 1.0, 0.0, 2, FAKE, FAKE, None, FAKE, FAKE, FAKE, FAKE,
                1 << 40, None) == -1
    assert C.sizeof(C.c_float) * len(B.SOLVE_FIELDS) == 16


def test_certificate_argument_validation(lib):
    ok = B.make_shape(2, 8, 2, 64, 256)
    s = C.byref(ok)
    r = lib.vsa_build_page_radii
    assert r(s, None, FAKE, FAKE, FAKE, None, FAKE, None) == -1
    assert r(s, FAKE, FAKE, FAKE, FAKE, None, None, None) == -1
    assert r(s, ODD, FAKE, FAKE, FAKE, None, FAKE, None) == -4
    step = lib.vsa_decode_step_certified

    def call(shape=ok, radii=FAKE, cert=FAKE, ws_bytes=1 << 40, P=4, K_c=16):
        return step(C.byref(shape), FAKE, FAKE, radii, FAKE, FAKE, FAKE, FAKE, P, K_c, 1.0, 0.0, FAKE, FAKE, cert, FAKE,
                    FAKE, FAKE, FAKE, ws_bytes, None)

    assert call(radii=None) == -1 and call(cert=None) == -1
    plain = B.vsa_workspace_bytes(ok, 4, 16, B.VSA_WS_STEP)
    need = B.vsa_workspace_bytes(ok, 4, 16, B.VSA_WS_STEP_CERTIFIED)
    assert need >= plain + 2 * 2 * 64 * 4            # + one fp32 radius per (sequence, kv head, logical page)
    assert call(ws_bytes=plain) == -3
    wide = B.make_shape(40, 8, 2, 9000, 1 << 16)     # 320 units > SMs: 256 threads hold at most 8192 page scores
    assert call(shape=wide) == -2
    exp = lib.vsa_decode_step_certified_expand

    def call_e(P=4, P2=8, K_c=16, ws_bytes=1 << 40, cert=FAKE):
        return exp(s, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, P, P2, K_c, 1.0, 0.0, FAKE, FAKE, cert, FAKE, FAKE, FAKE,
                   FAKE, ws_bytes, None)

    assert call_e(P2=4) == -1 and call_e(P2=3) == -1      # the expansion must add pages
    assert call_e(P2=129) == -2
    assert call_e(cert=None) == -1
    assert call_e(ws_bytes=B.vsa_workspace_bytes(ok, 4, 16, B.VSA_WS_STEP_CERTIFIED)) == -3
    assert B.vsa_workspace_bytes(ok, 8, 16, B.VSA_WS_STEP_EXPAND) >= need + 16 * 4
    assert C.sizeof(C.c_int32) * len(B.CERT_FIELDS) == 16


def test_append_argument_validation(lib):
    ok = B.make_shape(2, 8, 2, 64, 256)
    a = lib.vsa_append_kv
    assert a(C.byref(ok), None, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, None) == -1
    assert a(C.byref(ok), FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, None, None) == -1
    assert a(C.byref(ok), ODD, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, None) == -4
    assert a(None, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, None) == -1


def test_dense_and_step_argument_validation(lib):
    ok = B.make_shape(2, 8, 2, 64, 256)
    s = C.byref(ok)
    f = lib.vsa_dense_decode_fallback
    assert f(s, FAKE, FAKE, FAKE, FAKE, FAKE, None, FAKE, 1.0, FAKE, None, FAKE, 1 << 40, None) == -1  # count w/o list
    assert f(s, FAKE, FAKE, FAKE, FAKE, FAKE, None, None, 1.0, FAKE, None, FAKE, 16, None) == -3
    assert f(s, FAKE, FAKE, FAKE, FAKE, FAKE, None, None, 0.0, FAKE, None, FAKE, 1 << 40, None) == -1
    assert f(s, FAKE, FAKE, FAKE, FAKE, FAKE, None, None, 1.0, None, None, FAKE, 1 << 40, None) == -1
    g = lib.vsa_decode_step
    assert g(s, FAKE, None, FAKE, FAKE, FAKE, FAKE, 4, 16, 1.0, 0.0, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 1 << 40, None) == -1
    assert g(s, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 4, 16, 1.0, 0.0, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 64, None) == -3
    h = lib.vsa_decode_step_host
    assert h(s, None, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 4, 16, 1.0, 0.0, FAKE, FAKE, None, FAKE, FAKE, FAKE, FAKE,
             FAKE, 1 << 40, None) == -1
    assert h(s, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 4, 16, -2.0, 0.0, FAKE, FAKE, None, FAKE, FAKE, FAKE, FAKE,
             FAKE, 1 << 40, None) == -1
    b = lib.vsa_build_page_summaries
    assert b(s, None, FAKE, FAKE, None, FAKE, None) == -1
    assert b(s, FAKE, FAKE, FAKE, None, ODD, None) == -4


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "libvsa.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        B.lib()


def test_two_level_and_group_shared_argument_validation(lib):
    s = B.make_shape(8, 32, 8, 2048, 65536)
    sp = C.byref(s)
    # two-level routing: representatives, routing call, step
    assert lib.vsa_build_super_summaries(sp, None, FAKE, FAKE, None, FAKE, None, None) == -1
    assert lib.vsa_build_super_summaries(sp, FAKE, FAKE, FAKE, None, ODD, None, None) == -4
    route_ws = B.vsa_workspace_bytes(s, 32, 0, B.VSA_WS_ROUTE_TWO_LEVEL)
    assert route_ws > B.vsa_workspace_bytes(s, 32, 0, B.VSA_WS_ROUTE)
    assert B.vsa_workspace_bytes(s, 32, 256, B.VSA_WS_STEP_TWO_LEVEL) > route_ws
    assert B.vsa_workspace_bytes(s, 0, 0, B.VSA_WS_ROUTE_TWO_LEVEL) == 0

    def two(P_super=32, P=32, sup=FAKE, ws_bytes=1 << 40):
        return lib.vsa_route_pages_two_level(sp, FAKE, FAKE, sup, FAKE, FAKE, P_super, P, FAKE, None, None, FAKE,
                                             ws_bytes, None)
    assert two(sup=None) == -1 and two(P_super=0) == -1 and two(P_super=129) == -2 and two(P=0) == -1
    assert two(sup=ODD) == -4 and two(ws_bytes=route_ws - 1) == -3

    def two_step(K_c=256, eps=11.3, ws_bytes=1 << 40, P_super=32):
        return lib.vsa_decode_step_two_level(sp, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, P_super, 32, K_c, eps, 90.0,
                                             FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, ws_bytes, None)
    assert two_step(K_c=0) == -1 and two_step(K_c=513) == -2 and two_step(eps=0.0) == -1
    assert two_step(ws_bytes=1024) == -3 and two_step(P_super=0) == -1

    # group-shared step: shapes and layouts it refuses on the host
    def shared(shape, K_c=256, ws_bytes=1 << 40, q=FAKE):
        return lib.vsa_decode_step_group_shared(C.byref(shape), q, FAKE, FAKE, FAKE, FAKE, FAKE, 32, K_c, 11.3, 90.0,
                                                FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, ws_bytes, None)
    assert shared(s, K_c=0) == -1 and shared(s, q=None) == -1 and shared(s, q=ODD) == -4
    assert shared(s, ws_bytes=1024) == -3
    assert shared(B.make_shape(8, 32, 1, 2048, 65536)) == -2          # 32 query heads per KV head
    strided = B.make_shape(8, 32, 8, 2048, 65536)
    strided.kv_token_stride = 256                                      # rows not contiguous: no 4 KB tiles
    strided.kv_head_stride = 16 * 256
    strided.kv_page_stride = 8 * 16 * 256
    assert shared(strided) == -2


def test_multi_query_group_sizes_are_accepted(lib):
    for hq, hkv in ((16, 1), (32, 1), (32, 2)):
        s = B.make_shape(4, hq, hkv, 2048, 65536)
        assert B.vsa_workspace_bytes(s, 32, 256, B.VSA_WS_STEP) > 0
    assert B.vsa_workspace_bytes(B.make_shape(4, 48, 1, 2048, 65536), 32, 256, B.VSA_WS_STEP) == 0   # group of 48


def test_context_parallel_and_head_dimension_argument_validation(lib):
    s = B.make_shape(8, 32, 8, 2048, 65536)
    sp = C.byref(s)

    def cand(q=FAKE, P=32, K_out=257, pos=FAKE, shape=sp):
        return lib.vsa_cp_token_candidates(shape, q, FAKE, FAKE, FAKE, FAKE, P, K_out, pos, FAKE, None)
    assert cand(q=None) == -1 and cand(pos=None) == -1 and cand(K_out=0) == -1 and cand(P=0) == -1
    assert cand(P=129) == -2 and cand(P=2, K_out=34) == -2 and cand(q=ODD) == -4

    def readout(v=FAKE, K_c=256, eps=11.3, out=FAKE, shape=sp):
        return lib.vsa_cp_partial_readout(shape, v, FAKE, FAKE, FAKE, FAKE, K_c, eps, out, FAKE, None)
    assert readout(v=None) == -1 and readout(out=None) == -1 and readout(K_c=0) == -1 and readout(eps=0.0) == -1
    assert readout(K_c=4096) == -2 and readout(v=ODD) == -4
    # the sharded kernels and the variants beyond the closed-form step exist at head dimension 128 only
    for d in (64, 256):
        sd = B.make_shape(8, 32, 8, 2048, 65536, head_dim=d)
        assert cand(shape=C.byref(sd)) == -2 and readout(shape=C.byref(sd)) == -2
        assert lib.vsa_build_page_radii(C.byref(sd), FAKE, FAKE, FAKE, FAKE, None, FAKE, None) == -2
        assert lib.vsa_append_kv(C.byref(sd), FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, None) == -2
        assert lib.vsa_build_super_summaries(C.byref(sd), FAKE, FAKE, FAKE, None, FAKE, None, None) == -2
        assert B.vsa_workspace_bytes(sd, 32, 256, B.VSA_WS_STEP) > 0
    # 32-token pages: at most 64 routed pages (2048 scored tokens per unit)
    s32 = B.make_shape(8, 32, 8, 2048, 65536, page_size=32)
    assert lib.vsa_sparse_decode(C.byref(s32), FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, 65, 256, 11.3, 90.0, FAKE, FAKE, FAKE,
                                 FAKE, None, 0, None) == -2
