"""Host-only checks of the C-ABI library: it loads without a GPU, exports every symbol the header
declares, and rejects bad arguments with the documented codes before touching CUDA."""
import ctypes
import re
from pathlib import Path

import pytest

from paper_2609_39223_b200 import api

ROOT = Path(__file__).resolve().parent.parent
HEADER = (ROOT / "include" / "qf.h").read_text()
P = 0x10000            # a fake, 16-byte aligned, never dereferenced device address


def declared_symbols():
    return sorted(set(re.findall(r"\b(qf_[a-z0-9_]+)\s*\(", HEADER)) - {"qf_status_t", "qf_format_t"})


def test_library_exports_every_declared_symbol():
    L = api.lib()
    names = declared_symbols()
    assert len(names) >= 12
    for n in names:
        assert hasattr(L, n), n
    assert sorted(api.EXPORTS) == names


def test_no_torch_or_cxx_types_in_the_header():
    assert "torch" not in HEADER and "std::" not in HEADER and "at::" not in HEADER
    assert 'extern "C"' in HEADER


def test_header_is_plain_c99(tmp_path):
    """The boundary is a C ABI: the header must compile as strict C99 with nothing but the standard headers."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler on this machine")
    src = tmp_path / "use_qf.c"
    src.write_text('#include "qf.h"\nint main(void) { return qf_status_string(QF_OK) != 0 && sizeof(qf_format_t) > 0 ? 0 : 1; }\n')
    r = subprocess.run([gcc, "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror", "-I", str(ROOT / "include"), "-fsyntax-only", str(src)],
                       capture_output=True, text=True)
    assert r.returncode == 0, r.stderr


def test_version_and_status_strings():
    assert api.lib().qf_version() >= 100
    seen = {api.status_string(c) for c in range(10)}
    assert len(seen) == 10 and api.status_string(0) == "ok"
    assert "unknown" in api.status_string(99)


def test_workspace_bytes():
    f = api.qf_workspace_bytes
    assert f(api.OP_QDQ, 2048, 0, 2048) == 256
    M, N, K = 8192, 12288, 4096
    assert f(api.OP_LINEAR_FWD, M, N, K) == 256 + N * K * 2 + M * K * 2
    assert f(api.OP_GROUPED_FWD, 1024, 768, 2048, 128) == 256 + 128 * 768 * 2048 * 2 + 1024 * 2048 * 2
    assert f(api.OP_LINEAR_BWD, 1, 8, 16) % 256 == 0


def test_qdq_argument_errors_need_no_gpu():
    q = api.lib().qf_qdq
    big = 1 << 20
    assert q(9, P, 4, 64, P, P, P, P, 0, P, big, None) == 4                  # unknown format
    assert q(api.FMT_NONE, P, 4, 64, P, P, P, P, 0, P, big, None) == 4       # NONE is not a quantizer
    assert q(api.FMT_MXFP4, None, 4, 64, P, P, P, None, 0, P, big, None) == 1
    assert q(api.FMT_MXFP4, P, 4, 64, None, None, None, None, 0, P, big, None) == 1
    assert q(api.FMT_NVFP4, P, 4, 64, P, P, P, None, 0, P, big, None) == 1   # NVFP4 needs a tensor-scale slot
    assert q(api.FMT_MXFP4, P, 4, 48, P, P, P, None, 0, P, big, None) == 2   # 48 % 32 != 0
    assert q(api.FMT_NVFP4, P, 4, 40, P, P, P, P, 0, P, big, None) == 2
    assert q(api.FMT_Q4_K, P, 4, 128, P, P, P, None, 0, P, big, None) == 2
    assert q(api.FMT_MXFP4, P, -1, 64, P, P, P, None, 0, P, big, None) == 2
    assert q(api.FMT_MXFP4, P + 2, 4, 64, P, P, P, None, 0, P, big, None) == 3
    assert q(api.FMT_NVFP4, P, 4, 64, P, P, P, P, 0, None, 0, None) == 5     # amax pre-pass needs scratch
    assert q(api.FMT_NVFP4, P, 4, 64, P, P, P, P, 0, P, 16, None) == 5


def test_linear_argument_errors_need_no_gpu():
    L = api.lib()
    M, N, K = 128, 256, 512
    ws = api.qf_workspace_bytes(api.OP_LINEAR_FWD, M, N, K)
    fwd = lambda **kw: L.qf_fq_linear_fwd(kw.get("X", P), kw.get("W", P), kw.get("Y", P), kw.get("dt", 0), kw.get("M", M),
                                          kw.get("N", N), kw.get("K", K), kw.get("wq", 2), kw.get("aq", 2), None, None, None,
                                          kw.get("flags", 0), kw.get("ws", P), kw.get("wsb", ws), None)
    assert fwd(X=None) == 1
    assert fwd(dt=7) == 9
    assert fwd(aq=api.FMT_Q4_K) == 4                    # Q4_K is weight-only
    assert fwd(wq=5) == 4
    assert fwd(K=520) == 2                              # not a multiple of 32
    assert fwd(N=250) == 2
    assert fwd(wq=api.FMT_Q4_K, aq=0, K=512) != 2
    assert fwd(wq=api.FMT_Q4_K, aq=0, K=384) == 2
    assert fwd(Y=P + 8) == 3
    assert fwd(ws=None) == 5
    assert fwd(wsb=ws - 1) == 5
    assert fwd(wq=api.FMT_NVFP4, flags=api.W_TSCALE_GIVEN) == 1   # flag says "given" but no pointer
    bwd = L.qf_fq_linear_bwd
    assert bwd(P, P, P, None, 0, None, 0, M, N, K, 2, 2, None, None, 0, P, ws, None) == 1       # nothing requested
    assert bwd(None, P, P, P, 0, P, 1, M, N, K, 2, 2, None, None, 0, P, ws, None) == 1
    assert bwd(P, P, P, P, 3, P, 1, M, N, K, 2, 2, None, None, 0, P, ws, None) == 9
    g = L.qf_fq_grouped_linear_fwd
    assert g(P, P, P, 0, None, 4, 512, N, K, 2, 2, None, None, 0, P, 1 << 30, None) == 1
    assert g(P, P, P, 0, P, 4, 500, N, K, 2, 2, None, None, 0, P, 1 << 30, None) == 2          # rows not padded to 128
    assert g(P, P, P, 0, P, 0, 512, N, K, 2, 2, None, None, 0, P, 1 << 30, None) == 2
    # grouped NVFP4 weights need the per-expert scale array: refused with the other checks, before anything is enqueued
    assert g(P, P, P, 0, P, 4, 512, N, K, api.FMT_NVFP4, 0, None, None, 0, P, 1 << 30, None) == 1


def test_batched_argument_errors_need_no_gpu():
    L = api.lib()
    arr = lambda *v: (api.c_void_p * len(v))(*v)
    i64 = lambda *v: (api.c_int64 * len(v))(*v)
    call = lambda fmt, n, ins, rows, cols, outs, ts, ws, wsb: L.qf_qdq_batched(fmt, n, ins, rows, cols, outs, None, None, ts, 0, ws, wsb, None)
    assert call(api.FMT_MXFP4, -1, arr(P), i64(4), i64(64), arr(P), None, None, 0) == 2
    assert call(api.FMT_MXFP4, 0, None, None, None, None, None, None, 0) == 0
    assert call(api.FMT_MXFP4, 1, None, i64(4), i64(64), arr(P), None, None, 0) == 1
    assert call(api.FMT_MXFP4, 2, arr(P, P), i64(4, 4), i64(64, 48), arr(P, P), None, None, 0) == 2          # second tensor: bad cols
    assert call(api.FMT_MXFP4, 2, arr(P, P + 4), i64(4, 4), i64(64, 64), arr(P, P), None, None, 0) == 3      # second tensor: misaligned
    assert call(api.FMT_MXFP4, 1, arr(P), i64(4), i64(64), None, None, None, 0) == 1                          # no output at all
    assert call(api.FMT_NVFP4, 1, arr(P), i64(4), i64(64), arr(P), None, P, 1 << 20) == 1                     # NVFP4 needs the scale array
    assert call(api.FMT_NVFP4, 3, arr(P, P, P), i64(4, 4, 4), i64(64, 64, 64), arr(P, P, P), P, P, 256) == 5  # workspace too small
    assert api.qf_workspace_bytes(api.OP_QDQ_BATCHED, 0, 0, 0, 3) == 512


def test_calls_fail_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    big = 1 << 20
    # valid arguments, no GPU: the library reports a CUDA error instead of computing anything on the host
    assert api.lib().qf_qdq(api.FMT_MXFP4, P, 4, 64, P, P, P, None, 0, P, big, None) == 6
    with pytest.raises(Exception):
        api.qf_qdq(api.FMT_MXFP4, torch.zeros(4, 64, dtype=torch.bfloat16))
