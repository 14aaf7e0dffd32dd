"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every symbol the
public header declares, and its shape/size logic (no kernel launches) behaves as documented."""
import ctypes
import os
import re

import pytest

from paper_2608_12932_b200 import binding as B
from paper_2608_12932_b200 import build as libbuild
from paper_2608_12932_b200 import workload as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    libbuild.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "w4a8.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(w4a8_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = declared_functions()
    assert set(names) == set(B.EXPORTS)
    lib = ctypes.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n


def test_library_needs_no_driver_to_load():
    # libcuda is resolved lazily by the static runtime, so loading works on a CPU-only host
    out = os.popen(f"ldd {B.LIB_PATH}").read()
    assert "libcuda.so" not in out and "libcudart" not in out


def test_size_queries():
    for (K, N) in wl.LAYERS.values():
        G = K // 128
        assert B.w4a8_packed_bytes(N, K) == N * K // 2 + G * N * 5 // 2
        assert B.w4a8_workspace_bytes(0, N, K) == B.WORKSPACE_HEADER_BYTES
        w8, w16, w64, w4096 = (B.w4a8_workspace_bytes(m, N, K) for m in (8, 16, 64, 4096))
        assert B.WORKSPACE_ZEROED_BYTES < w8 < w16 < w64 <= w4096
        # after the header: one hand-over slot per CTA of the strip kernel (a strip of at most 128 channels x 16 tokens,
        # a float and a tag per sum), zero between calls; then the split-K slices / hand-over tiles of the other kernels
        assert B.WORKSPACE_ZEROED_BYTES == B.WORKSPACE_HEADER_BYTES + 192 * 128 * 16 * 8
        # from 17 tokens on the tensor-core kernel may need its hand-over area (one fp32 tile per CTA)
        assert w4096 >= B.WORKSPACE_HEADER_BYTES + 148 * 208 * 128 * 4
        assert (w64 - B.WORKSPACE_ZEROED_BYTES) % (64 * N * 4) == 0
    assert B.w4a8_packed_bytes(100, 256) == 0
    assert B.w4a8_packed_bytes(128, 100) == 0
    assert B.w4a8_packed_bytes(128, 256, 64) == 0
    assert B.w4a8_workspace_bytes(8, 128, 256, 32) == 0
    assert B.w4a8_workspace_bytes(-1, 128, 256) == 0
    assert B.w4a8_packed_bytes(128 * 961, 128) == 0          # more tiles than the workspace header has counters


def test_plan_query_invariants():
    """w4a8_plan is host-only: on a machine without a GPU it assumes 148 SMs and no cluster occupancy
    (so no K split of the tensor-core kernel), and its answers obey the dispatch rules."""
    sms = 148
    for (K, N) in list(wl.LAYERS.values()) + [(256, 256), (1024, 384), (3072, 256)]:
        tiles, G = N // 128, K // 128
        for M in (1, 7, 8, 9, 16, 17, 32, 33, 64, 65, 128, 200, 256, 512, 1024, 4096):
            p = B.w4a8_plan(M, N, K)
            assert p["family"] in (B.PATH_STRIP, B.PATH_SPLITK, B.PATH_TCGEN05)
            if M <= 16:
                assert p["family"] in (B.PATH_STRIP, B.PATH_SPLITK)
            if M > 64:
                assert p["family"] == B.PATH_TCGEN05
            if p["family"] == B.PATH_STRIP:
                # at most two CTAs per SM, one strip per CTA at least (a strip is shared by at most two CTAs); never a K split
                R = p["strip_rows"]
                assert R in (16, 32, 64, 128) and p["k_slices"] == 1 and p["tile_m"] == (8 if M <= 8 else 16)
                assert 1 <= p["ctas"] <= min(2 * sms, N // R)
                assert p["balanced"] == int((N // R) % p["ctas"] != 0)
                if M > 8:
                    assert R == 32
                else:
                    # the widest strip that keeps about 1.25 strips per SM, one step narrower if that leaves fewer than two per SM
                    assert R == 16 or N // R >= (sms * 5) // 4
                    assert R >= 64 or N // (2 * R) < (sms * 5) // 4 or (R == 32 and N // 64 < 2 * sms)
            elif p["family"] == B.PATH_SPLITK:
                assert p["strip_rows"] == 0
                assert p["tile_m"] in (8, 16, 32, 64) and p["tile_m"] >= min(M, 64)
                assert 1 <= p["k_slices"] <= min(8, G) and p["ctas"] == tiles * p["k_slices"] and p["balanced"] == 0
            else:
                assert p["tile_m"] in (64, 128, 208) and 1 <= p["k_slices"] <= 4
                all_tiles = -(-M // p["tile_m"]) * tiles
                if p["k_slices"] > 1:
                    assert p["ctas"] == all_tiles * p["k_slices"] <= sms and G // p["k_slices"] >= 4
                else:
                    assert p["ctas"] == min(all_tiles, sms)
                # the balanced walk only where there are more tiles than CTAs that do not divide evenly, never with a K split
                assert p["balanced"] in (0, 1)
                if p["balanced"]:
                    assert p["k_slices"] == 1 and all_tiles > sms and all_tiles % sms != 0
                # never a taller tile than the next height down that already covers M
                assert not (p["tile_m"] == 208 and M <= 128) and not (p["tile_m"] == 128 and M <= 64)
    # several waves of tiles: the tallest tile; a bad shape: an error
    assert B.w4a8_plan(4096, 24576, 4096)["tile_m"] == 208
    # long K and 160 tiles on 148 SMs: the balanced walk (two rounds of whole tiles would leave most SMs idle half the time)
    assert B.w4a8_plan(1024, 4096, 12288)["balanced"] == 1
    assert B.w4a8_plan(4096, 24576, 4096)["balanced"] == 0
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_plan(8, 100, 256)
    assert e.value.code == B.ERR_SHAPE
    with pytest.raises(B.W4A8Error):
        B.w4a8_plan(0, 256, 256)


def test_status_strings():
    seen = {B.status_string(c) for c in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert B.status_string(99) == "unknown status"


def test_shape_validation_needs_no_gpu():
    L = B.lib()
    # shape errors are reported before any CUDA call
    assert L.w4a8_quantize_act(None, 4, 200, 128, None, None, None, None) == B.ERR_SHAPE
    assert L.w4a8_quantize_act(None, -1, 256, 128, None, None, None, None) == B.ERR_SHAPE
    assert L.w4a8_quantize_act(None, 0, 256, 128, None, None, None, None) == B.OK
    assert L.w4a8_quantize_act(None, 4, 256, 128, None, None, None, None) == B.ERR_NULL
    assert L.w4a8_pack_weights(None, None, None, 100, 256, 128, None, None) == B.ERR_SHAPE
    assert L.w4a8_pack_weights(None, None, None, 128, 256, 128, None, None) == B.ERR_NULL
    assert L.w4a8_gemm(None, None, None, None, None, 8, 128, 256, 64, None, 0, None, None) == B.ERR_SHAPE
    assert L.w4a8_gemm(None, None, None, None, None, 0, 128, 256, 128, None, 0, None, None) == B.OK
    assert L.w4a8_gemm(None, None, None, None, None, 8, 128, 256, 128, None, 0, None, None) == B.ERR_NULL
    assert L.w4a8_gemm_path(9, None, None, None, None, None, 8, 128, 256, 128, None, 0, None, None) == B.ERR_SHAPE
    assert L.w4a8_gemm_path(B.PATH_SPLITK, None, None, None, None, None, 65, 128, 256, 128, None, 0, None, None) == B.ERR_SHAPE
    assert L.w4a8_gemm_path(B.PATH_SPLITK_WORKSPACE, None, None, None, None, None, 65, 128, 256, 128, None, 0, None, None) == B.ERR_SHAPE
    assert L.w4a8_gemm_static_scratch(None, None, None, None, None, 65, 128, 256, 128, None) == B.ERR_SHAPE
    assert L.w4a8_gemm_static_scratch(None, None, None, None, None, 8, 128, 256, 128, None) == B.ERR_NULL
    assert L.w4a8_gemm_per_channel(None, None, None, None, 8, 128, 256, 64, None, 0, None, None) == B.ERR_SHAPE
    assert L.w4a8_gemm_per_channel(None, None, None, None, 8, 128, (1 << 19) + 128, 128, None, 0, None, None) == B.ERR_SHAPE
    assert L.w4a8_gemm_per_channel(None, None, None, None, 0, 128, 256, 128, None, 0, None, None) == B.OK
    assert L.w4a8_gemm_per_channel(None, None, None, None, 8, 128, 256, 128, None, 0, None, None) == B.ERR_NULL
    assert L.w4a8_workspace_init(None, 4096, None) == B.ERR_NULL
    assert L.w4a8_check_status(None, None) == B.ERR_NULL
    # alignment is checked before the device is queried
    assert L.w4a8_quantize_act(ctypes.c_void_p(0x1002), 4, 256, 128, ctypes.c_void_p(0x2000),
                               ctypes.c_void_p(0x3000), ctypes.c_void_p(0x4000), None) == B.ERR_ALIGN


def test_misaligned_output_is_refused_without_a_gpu():
    """The GEMM kernels store y in 8- and 16-byte pieces, so a bf16 view that starts one element into a
    buffer must come back as ERR_ALIGN.  Alignment is checked before the device is touched: the pointers
    below are made-up numbers and nothing is launched."""
    L = B.lib()
    vp = ctypes.c_void_p
    qa, sa, asum, pw, ws = vp(0x10000), vp(0x20000), vp(0x30000), vp(0x40000), vp(0x50000)
    big = 1 << 30
    for bad_y in (0x60002, 0x60008):
        assert L.w4a8_gemm(qa, sa, asum, pw, vp(bad_y), 8, 128, 256, 128, ws, big, None, None) == B.ERR_ALIGN
        for path in (B.PATH_AUTO, B.PATH_SPLITK, B.PATH_TCGEN05):
            assert L.w4a8_gemm_path(path, qa, sa, asum, pw, vp(bad_y), 8, 128, 256, 128, ws, big, None, None) == B.ERR_ALIGN
        assert L.w4a8_gemm_per_channel(qa, sa, pw, vp(bad_y), 8, 128, 256, 128, ws, big, None, None) == B.ERR_ALIGN
        assert L.w4a8_linear(vp(0x70000), pw, vp(bad_y), 8, 128, 256, 128, qa, sa, asum, ws, big, None) == B.ERR_ALIGN
        assert L.w4a8_linear_host(vp(0x80000), vp(0x90000), 8, 128, 256, 128, pw, vp(0x70000), qa, sa, asum,
                                  vp(bad_y), ws, big, None) == B.ERR_ALIGN
    # the element-by-element kernels take any bf16 pointer: the next check (workspace size) is what refuses this call
    assert L.w4a8_gemm_path(B.PATH_SPLITK_WORKSPACE, qa, sa, asum, pw, vp(0x60002), 8, 128, 256, 128, ws, 0, None,
                            None) == B.ERR_WORKSPACE
    # a misaligned static-scratch call is refused the same way
    assert L.w4a8_gemm_static_scratch(qa, sa, asum, pw, vp(0x60001), 8, 128, 256, 128, None) == B.ERR_ALIGN


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        B.lib()
