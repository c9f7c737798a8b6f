"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and its host
logic (storage planner, argument validation that happens before any device work) behaves."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import synth_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2502_08141_b200 import build
    build.build()
    import paper_2502_08141_b200 as lw
    return lw


def test_library_exports_every_declared_symbol(lib):
    import glob
    header = "".join(open(h).read() for h in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))))
    declared = set(re.findall(r"\b(lowra_[a-z_]+)\s*\(", header))
    assert declared == set(lib.EXPORTS)
    L = lib.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_status_strings(lib):
    assert lib.status_string(0) == "ok"
    assert len({lib.status_string(c) for c in range(10)}) == 10


def test_plan_matches_oracle_layout(lib):
    for N, K, mix, mid in ((1000, 256, {1: 0.3, 2: 0.5, 4: 0.2}, 1), (77, 128, {4: 1.0}, 2),
                           (512, 512, {1: 0.5, 2: 0.5}, 3), (5, 1280, {2: 1.0}, 4)):
        precs = si.precisions(N, mix, matrix_id=mid)
        got = lib.lowra_plan(precs, K)
        want = oracle.plan(precs, K)
        assert np.array_equal(got["perm"], want["perm"])
        assert np.array_equal(got["inv_perm"], want["inv_perm"])
        assert got["counts"] == list(want["counts"])
        assert got["seg_off"] == [int(x) for x in want["seg_off"]]
        assert got["packed_bytes"] == want["packed_bytes"] == sum(K * int(b) // 8 for b in precs)


def test_plan_rejects_bad_input(lib):
    with pytest.raises(lib.LowraError) as e:
        lib.lowra_plan(np.array([1, 2, 3], np.uint8), 128)
    assert e.value.code == lib.LOWRA_ERR_PREC
    with pytest.raises(lib.LowraError) as e:
        lib.lowra_plan(np.array([1, 2, 4], np.uint8), 100)
    assert e.value.code == lib.LOWRA_ERR_SHAPE
    with pytest.raises(lib.LowraError) as e:
        lib.lowra_plan(np.zeros(0, np.uint8), 128)
    assert e.value.code == lib.LOWRA_ERR_SHAPE


def test_validation_runs_before_any_device_work(lib):
    """Null pointers / bad shapes are refused on the host, so this needs no GPU."""
    L = lib.lib()
    lay = lib._CLayout()
    lay.N, lay.K, lay.block = 8, 128, 64
    lay.counts[0] = 8
    lay.packed_bytes = 8 * 128 // 8
    lay.seg_off[1] = lay.seg_off[2] = lay.packed_bytes
    # null device arrays in the layout
    assert L.lowra_decode(ctypes.byref(lay), None, None, None, None, None) == lib.LOWRA_ERR_NULL
    lay.precs_dev = lay.perm_dev = lay.inv_perm_dev = 4096   # fake, never dereferenced
    assert L.lowra_decode(ctypes.byref(lay), None, None, None, None, None) == lib.LOWRA_ERR_NULL
    assert L.lowra_encode(ctypes.byref(lay), 4096, 4096, 4096 + 8, 4096, None) == lib.LOWRA_ERR_ALIGN
    lay.block = 32
    assert L.lowra_decode(ctypes.byref(lay), 4096, 4096, 4096, 4096, None) == lib.LOWRA_ERR_SHAPE
    lay.block = 64
    lay.counts[0] = 7
    assert L.lowra_decode(ctypes.byref(lay), 4096, 4096, 4096, 4096, None) == lib.LOWRA_ERR_PREC
    lay.counts[0] = 8
    assert L.lowra_workspace_bytes(ctypes.byref(lay), 16, 16) > 256
    assert L.lowra_workspace_bytes(ctypes.byref(lay), 16, 24) == 0      # rank must be a multiple of 16
    assert L.lowra_workspace_bytes(ctypes.byref(lay), 0, 16) == 0
    args = [ctypes.byref(lay), 4096, 4096, 4096, 4096, 16, 4096, 4096, 24, ctypes.c_float(1.0), 4096, 4096, 1 << 20, None]
    assert L.lowra_lora_forward(*args) == lib.LOWRA_ERR_SHAPE
    args[8] = 16
    args[12] = 16                                                        # workspace too small
    assert L.lowra_lora_forward(*args) == lib.LOWRA_ERR_WORKSPACE
    assert L.lowra_lora_backward_input(*args) == lib.LOWRA_ERR_WORKSPACE
    assert L.lowra_device_status(None, None) == lib.LOWRA_ERR_NULL
    # a deal kept by the caller and the workspace initialisation that goes with it
    assert L.lowra_deal_bytes(None) == 0
    need_deal = L.lowra_deal_bytes(ctypes.byref(lay))
    assert need_deal >= 8 * 4 and need_deal % 256 == 0
    assert L.lowra_deal_build(ctypes.byref(lay), None, need_deal, None) == lib.LOWRA_ERR_NULL
    assert L.lowra_deal_build(ctypes.byref(lay), 4096 + 16, need_deal, None) == lib.LOWRA_ERR_ALIGN
    assert L.lowra_deal_build(ctypes.byref(lay), 4096, need_deal - 1, None) == lib.LOWRA_ERR_WORKSPACE
    assert L.lowra_deal_build(None, 4096, need_deal, None) == lib.LOWRA_ERR_NULL
    assert L.lowra_workspace_init(None, 1 << 20, None) == lib.LOWRA_ERR_NULL
    assert L.lowra_workspace_init(4096, 16, None) == lib.LOWRA_ERR_WORKSPACE
    assert L.lowra_workspace_init(4096 + 16, 1 << 20, None) == lib.LOWRA_ERR_WORKSPACE
    lay.deal_dev = 4096 + 16                                             # a deal that is not 256-byte aligned
    args[12] = 1 << 30
    assert L.lowra_lora_forward(*args) == lib.LOWRA_ERR_ALIGN
    lay.deal_dev = None
    args[12] = 16
    sargs = [ctypes.byref(lay), 4096, 4096, 4096, 4096, 1 << 20, 4096, 4096, 128, ctypes.c_float(1.0), 4096, None, None]
    assert L.lowra_lora_forward_static(*sargs) == lib.LOWRA_ERR_LIMIT   # 1M tokens x rank 128 needs > 8 MiB of scratch
    sargs[8] = 24
    assert L.lowra_lora_forward_static(*sargs) == lib.LOWRA_ERR_SHAPE
    assert L.lowra_dense_nt(4096, 4096, 16, 16, 100, 4096, 4096, 256, None) == lib.LOWRA_ERR_SHAPE
    assert L.lowra_dense_nt(4096, None, 16, 16, 128, 4096, 4096, 256, None) == lib.LOWRA_ERR_NULL
    init = (ctypes.c_double * 48)()
    assert L.lowra_learn_codebooks(ctypes.byref(lay), 4096, None, init, 10, 4096, 4096, None) == lib.LOWRA_ERR_NULL
    assert L.lowra_learn_codebooks(ctypes.byref(lay), 4096, init, init, -1, 4096, 4096, None) == lib.LOWRA_ERR_SHAPE
    assert L.lowra_learn_codebooks(ctypes.byref(lay), 4096 + 4, init, init, 10, 4096, 4096, None) == lib.LOWRA_ERR_ALIGN
    assert L.lowra_learn_codebooks_all(16, 256, 4096, init, None, 10, 4096, 4096, None) == lib.LOWRA_ERR_NULL
    assert L.lowra_learn_codebooks_all(16, 200, 4096, init, init, 10, 4096, 4096, None) == lib.LOWRA_ERR_SHAPE
    assert L.lowra_learn_codebooks_all(0, 256, 4096, init, init, 10, 4096, 4096, None) == lib.LOWRA_ERR_SHAPE
    assert L.lowra_learn_codebooks_all(16, 256, 4096, init, init, 10, 4096 + 4, 4096, None) == lib.LOWRA_ERR_ALIGN
    # natural-order offsets (host only) and the row reordering
    import numpy as np
    pr = np.array([1, 4, 2, 2], dtype=np.uint8)
    off = np.zeros(5, dtype=np.uint64)
    assert L.lowra_natural_offsets(4, 256, pr.ctypes.data, off.ctypes.data) == lib.LOWRA_OK
    assert off.tolist() == [0, 32, 160, 224, 288]
    assert L.lowra_natural_offsets(4, 200, pr.ctypes.data, off.ctypes.data) == lib.LOWRA_ERR_SHAPE
    pr[1] = 3
    assert L.lowra_natural_offsets(4, 256, pr.ctypes.data, off.ctypes.data) == lib.LOWRA_ERR_PREC
    assert L.lowra_natural_offsets(4, 256, None, off.ctypes.data) == lib.LOWRA_ERR_NULL
    assert L.lowra_reorder_rows(ctypes.byref(lay), 1, None, 4096, 4096, 8192, 8192, None) == lib.LOWRA_ERR_NULL
    assert L.lowra_reorder_rows(ctypes.byref(lay), 1, 4096, 4096, 4096, 4096, 8192, None) == lib.LOWRA_ERR_SHAPE
    assert L.lowra_reorder_rows(ctypes.byref(lay), 1, 4096, 4096 + 8, 4096, 8192, 8192, None) == lib.LOWRA_ERR_ALIGN
    # quantisation error: layout, W, maps, thresholds, sse, residual (may be NULL), stream
    assert L.lowra_quant_error(ctypes.byref(lay), 4096, 4096, 4096, None, None, None) == lib.LOWRA_ERR_NULL
    assert L.lowra_quant_error(ctypes.byref(lay), 4096 + 4, 4096, 4096, 4096, None, None) == lib.LOWRA_ERR_ALIGN
    assert L.lowra_quant_error(ctypes.byref(lay), 4096, 4096, 4096, 4096, 4096 + 8, None) == lib.LOWRA_ERR_ALIGN
    assert L.lowra_quant_error(None, 4096, 4096, 4096, 4096, None, None) == lib.LOWRA_ERR_NULL
    assert L.lowra_channel_errors(16, 256, 4096, 4096, 4096, None, None) == lib.LOWRA_ERR_NULL
    assert L.lowra_channel_errors(16, 200, 4096, 4096, 4096, 4096, None) == lib.LOWRA_ERR_SHAPE
    assert L.lowra_channel_errors(0, 256, 4096, 4096, 4096, 4096, None) == lib.LOWRA_ERR_SHAPE
    assert L.lowra_channel_errors(16, 256, 4096 + 4, 4096, 4096, 4096, None) == lib.LOWRA_ERR_ALIGN
    # adapter gradients: X, dY, M, K, N, A, B, r, s, dA, dB, workspace, bytes, stream
    big = 1 << 30
    assert L.lowra_adapter_workspace_bytes(0, 16) == 0
    assert L.lowra_adapter_workspace_bytes(16, 20) == 0
    need = L.lowra_adapter_workspace_bytes(300, 48)
    assert need >= 256 + 2 * 300 * 64 * 2
    ok = [4096, 4096, 300, 256, 512, 4096, 4096, 48, ctypes.c_float(1.0), 4096, 4096, 4096, big, None]
    def call(**kw):
        a = list(ok)
        for i, v in kw.items():
            a[int(i[1:])] = v
        return L.lowra_lora_backward_adapters(*a)
    assert call(_0=None) == lib.LOWRA_ERR_NULL
    assert call(_10=None) == lib.LOWRA_ERR_NULL
    assert call(_2=0) == lib.LOWRA_ERR_SHAPE
    assert call(_3=100) == lib.LOWRA_ERR_SHAPE       # K not a multiple of 8
    assert call(_7=8) == lib.LOWRA_ERR_SHAPE
    assert call(_5=4096 + 2) == lib.LOWRA_ERR_ALIGN
    assert call(_12=need - 1) == lib.LOWRA_ERR_WORKSPACE
    assert call(_11=4096 + 16) == lib.LOWRA_ERR_WORKSPACE
    lay.K = 128 * 400                                                    # a row no longer fits into shared memory
    lay.packed_bytes = 8 * lay.K // 8
    lay.seg_off[1] = lay.seg_off[2] = lay.packed_bytes
    assert L.lowra_learn_codebooks(ctypes.byref(lay), 4096, init, init, 10, 4096, 4096, None) == lib.LOWRA_ERR_SHAPE


def test_missing_library_fails_loudly(lib, monkeypatch, tmp_path):
    monkeypatch.setattr(lib, "_lib", None)
    monkeypatch.setattr(lib, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        lib.lib()


def test_public_headers_compile_as_plain_c(tmp_path):
    """The boundary is a C ABI: both headers must go through a C99 compiler on their own (no C++ in the signatures)."""
    import shutil
    import subprocess

    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "h.c"
    src.write_text('#include "lowra.h"\n#include "lowra_diag.h"\n'
                   "int main(void) { lowra_layout l; lowra_member m; lowra_group_member g; (void)l; (void)m; (void)g; return 0; }\n")
    out = subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(root, "include"),
                          "-c", str(src), "-o", str(tmp_path / "h.o")], capture_output=True, text=True)
    assert out.returncode == 0, out.stderr
