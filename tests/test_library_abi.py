"""The shared library builds for sm_100a, loads, exports every symbol that include/rdk.h declares,
and turns bad arguments into error codes on the host (nothing here launches a kernel)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2506_03206_b200 import build
    build.build()
    from paper_2506_03206_b200 import binding
    return binding


def test_header_symbols_are_exported(B):
    with open(os.path.join(ROOT, "include", "rdk.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    declared = set(re.findall(r"\b(rdk_[a-z_]+)\s*\(", text))
    assert declared == set(B.EXPORTS)
    L = B.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert B.rdk_version() >= 1000
    assert L.rdk_status_string(0) == b"ok" and L.rdk_status_string(3).startswith(b"no kept id")


def test_struct_layouts_match_the_header(B):
    assert C.sizeof(B.rdk_problem) == 56 and C.sizeof(B.rdk_affinity) == 24
    assert C.sizeof(B.rdk_outputs) == 10 * C.sizeof(C.c_void_p)


def test_size_queries(B):
    L = B.lib()
    assert L.rdk_kept_index_bytes(0, 4) == 0 and L.rdk_kept_index_bytes(16, 0) == 0
    a, b = L.rdk_kept_index_bytes(128256, 32064), L.rdk_kept_index_bytes(262144, 32768)
    assert 0 < a < b and a % 256 == 0
    assert L.rdk_build_affinity_workspace_bytes(1024, 256, 64) >= 1024 * 64 * 4
    pb = B.rdk_problem()
    pb.N, pb.n, pb.batch, pb.positions = 1024, 256, 2, 3
    assert L.rdk_exact_workspace_bytes(C.byref(pb), B.RDK_AFF_F32_ROWS) >= 6 * 256 * 4
    assert L.rdk_exact_workspace_bytes(C.byref(pb), B.RDK_AFF_BF16_COLS) >= 6 * 256 * 2
    assert L.rdk_exact_workspace_bytes(C.byref(pb), 7) == 0


def test_argument_errors_are_reported_on_the_host(B):
    L = B.lib()
    pb = B.rdk_problem()
    pb.N, pb.n, pb.batch, pb.positions = 0, 4, 1, 1
    out = B.rdk_outputs()
    dummy = C.c_void_p(256)
    st = L.rdk_sample_and_verify(C.byref(pb), 0, dummy, dummy, None, 0, dummy, 1, C.byref(out), None, 0, None)
    assert st == B.RDK_ERR_INVALID_ARG and b"positive" in L.rdk_last_error()
    pb.N = 16
    st = L.rdk_sample_and_verify(C.byref(pb), 0, dummy, dummy, None, 0, dummy, 1, C.byref(out), None, 0, None)
    assert st == B.RDK_ERR_INVALID_ARG          # kept_index is NULL
    pb.kept_index = 256
    st = L.rdk_sample_and_verify(C.byref(pb), 5, dummy, dummy, None, 0, dummy, 1, C.byref(out), None, 0, None)
    assert st == B.RDK_ERR_INVALID_ARG          # unknown mode
    st = L.rdk_sample_and_verify(C.byref(pb), 0, dummy, dummy, None, 0, dummy, 0, C.byref(out), None, 0, None)
    assert st == B.RDK_ERR_INVALID_ARG          # trials < 1
    st = L.rdk_sample_and_verify(C.byref(pb), 1, dummy, None, None, 0, dummy, 1, C.byref(out), None, 0, None)
    assert st == B.RDK_ERR_INVALID_ARG          # precomputed mode without w
    st = L.rdk_sample_and_verify(C.byref(pb), 0, dummy, dummy, None, 0, dummy, 1, C.byref(out), None, 0, None)
    assert st == B.RDK_ERR_WORKSPACE_TOO_SMALL  # the linear mode needs its workspace
    assert L.rdk_sample_workspace_bytes(C.byref(pb), 0, 1) >= 2112 and L.rdk_sample_workspace_bytes(C.byref(pb), 1, 1) == 0
    pb.target_dtype = 9
    st = L.rdk_sample_and_verify(C.byref(pb), 0, dummy, dummy, None, 0, dummy, 1, C.byref(out), None, 0, None)
    assert st == B.RDK_ERR_INVALID_ARG
    pb.target_dtype = 0
    pb.N = (1 << 21) + 1
    st = L.rdk_redistribute_linear(C.byref(pb), dummy, dummy, dummy, None, None, None)
    assert st == B.RDK_ERR_UNSUPPORTED
    pb.N = 16
    pb.target_row_stride = 8
    st = L.rdk_redistribute_linear(C.byref(pb), dummy, dummy, dummy, None, None, None)
    assert st == B.RDK_ERR_INVALID_ARG          # stride smaller than the row
    st = L.rdk_prepare_ids(None, 4, 16, dummy, 1 << 20, None, None)
    assert st == B.RDK_ERR_INVALID_ARG
    st = L.rdk_prepare_ids(dummy, 4, 16, dummy, 8, None, None)
    assert st == B.RDK_ERR_WORKSPACE_TOO_SMALL
    aff = B.rdk_affinity()
    aff.layout, aff.ld = B.RDK_AFF_BF16_COLS, 12            # ld not a multiple of 8
    st = L.rdk_build_affinity(dummy, 0, 8, 0, dummy, 4, 16, 0.1, C.byref(aff), dummy, dummy, 1 << 20, None)
    assert st == B.RDK_ERR_INVALID_ARG
    aff.layout, aff.ld = B.RDK_AFF_F32_ROWS, 16
    st = L.rdk_build_affinity(dummy, 0, 8, 0, dummy, 4, 16, 0.0, C.byref(aff), dummy, dummy, 1 << 20, None)
    assert st == B.RDK_ERR_INVALID_ARG          # tau must be positive
    st = L.rdk_build_affinity(dummy, 0, 8, 0, dummy, 4, 16, 0.1, C.byref(aff), dummy, dummy, 16, None)
    assert st == B.RDK_ERR_WORKSPACE_TOO_SMALL


def test_route_query_reports_host_side_argument_errors(B):
    L = B.lib()
    pb = B.rdk_problem()
    pb.N, pb.n, pb.batch, pb.positions = 0, 4, 1, 1
    why = C.c_char_p()
    assert L.rdk_sample_route(C.byref(pb), 0, None, None, 1, None, 0, C.byref(why)) == -B.RDK_ERR_INVALID_ARG
    pb.N, pb.kept_index = 8192, 256
    pb.target_dtype = pb.drafter_dtype = B.RDK_BF16
    # a precomputed w never streams; nor does a problem whose flags ask for the row kernel
    assert L.rdk_sample_route(C.byref(pb), 1, None, None, 1, None, 0, C.byref(why)) == B.RDK_ROUTE_ROW_KERNEL
    pb.flags = B.RDK_FLAG_ROW_KERNEL
    assert L.rdk_sample_route(C.byref(pb), 0, None, None, 1, None, 0, C.byref(why)) == B.RDK_ROUTE_ROW_KERNEL
    assert b"RDK_FLAG_ROW_KERNEL" in why.value
    pb.flags = B.RDK_FLAG_W_AS_GIVEN          # belongs to the precomputed-w mode only
    assert L.rdk_sample_route(C.byref(pb), 0, None, None, 1, None, 0, None) == -B.RDK_ERR_INVALID_ARG
    assert L.rdk_sample_route(C.byref(pb), 1, None, None, 1, None, 0, None) == B.RDK_ROUTE_ROW_KERNEL
    pb.flags = 4                              # not a flag
    assert L.rdk_sample_route(C.byref(pb), 0, None, None, 1, None, 0, None) == -B.RDK_ERR_INVALID_ARG
    # an index this process never prepared at that address: not known to be ascending
    pb.flags = 0
    dummy = C.c_void_p(4096)
    assert L.rdk_sample_route(C.byref(pb), 0, dummy, dummy, 1, dummy, 1 << 30, C.byref(why)) == B.RDK_ROUTE_ROW_KERNEL
    assert b"kept ids" in why.value


def test_binding_refuses_wrong_tensor_types(B):
    import torch
    with pytest.raises(TypeError):
        B.rdk_prepare_ids(torch.zeros(4, dtype=torch.int64), 16)
    with pytest.raises(TypeError):
        B._dtype_code(torch.zeros(2, dtype=torch.float16))


def test_stream_geometry_covers_the_vocabulary_and_fits_shared_memory(B):
    """Host logic of the streaming kernels' planner: for many shapes the segments cover the vocabulary,
    there are at most 256 of them, a segment is a whole number of 16-byte vectors per lane, the cache
    has room for the expected kept tokens of a warp, and the shared memory stays within one SM's."""
    import paper_2506_03206_b200 as rdk
    shapes = [(4096, 1), (4096, 4096), (4097, 100), (12808, 2000), (40000, 9000), (128256, 32064), (128256, 12826),
              (200000, 500), (262144, 32768), (262144, 262144), (400000, 50000)]
    for N, n in shapes:
        for tz, ty in ((B.RDK_BF16, B.RDK_BF16), (B.RDK_F32, B.RDK_F32), (B.RDK_BF16, B.RDK_F32)):
            g = rdk.rdk_stream_geometry(N, n, tz, ty)
            if not g["supported"]:
                continue
            per_vec = 32 * (8 if tz == B.RDK_BF16 else 4)
            assert g["segment_tokens"] % per_vec == 0
            segs = g["ctas_per_row"] * g["warps_per_cta"]
            assert segs * g["segment_tokens"] >= N and segs <= 256 and 1 <= g["ctas_per_row"] <= 16
            assert (segs - g["warps_per_cta"]) * g["segment_tokens"] < N            # the last CTA is not idle
            assert 2 <= g["stages"] <= 4 and 3 <= g["live_rows"] <= 8
            assert g["cached_slots_per_warp"] % 64 == 0 and g["cached_slots_per_warp"] >= 64
            assert g["dynamic_shared_bytes"] <= 212 * 1024
    big = rdk.rdk_stream_geometry(128256, 32064)
    assert big["ctas_per_row"] == 8 and big["segment_tokens"] == 1024      # the benchmark shape
    # bf16 logits with the common segment length keep the pair cache in tensor memory: 128 columns per
    # warp at 4 per 64-slot step and live row, so shared memory holds stages only
    assert big["live_rows"] * (big["cached_slots_per_warp"] // 64) * 4 <= 128 and big["stages"] >= 3
    assert rdk.rdk_stream_geometry(1000, 10)["supported"] == 0              # small vocabularies take the row kernel
    assert rdk.rdk_stream_geometry(1 << 21, 1000)["supported"] == 0         # too large for shared memory
