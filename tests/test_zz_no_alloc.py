"""The allocation-free forward entry point. Some hosts cannot give the library scratch memory when they
call it: an extension running inside a process whose memory planner took the whole device up front and
forbids further device allocations, or a loop that must never enter an allocator. For them the two
transient fake-quantized copies live in a fixed buffer inside the library. The entry point must give
exactly what the ordinary one gives, call after call, and must leave the amount of free device memory
untouched. Collected last on purpose; passes on its own and after the rest of the suite."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39223_b200 import api, synth
from util import torch_to_bits

TOL = 1e-2          # the linear-layer bound used everywhere: max|diff| <= 1e-2 * rms(reference)


@pytest.mark.gpu
def test_noalloc_forward_matches_workspace_forward_twice_in_a_row():
    M, N, K = 384, 520, 1024
    c1 = synth.linear_case(M, N, K, seed=21, outlier_channels=2)
    c2 = synth.linear_case(M, N, K, seed=22, outlier_channels=2)
    for wq, aq in ((api.FMT_MXFP4, api.FMT_MXFP4), (api.FMT_NVFP4, api.FMT_NVFP4)):
        for c in (c1, c2):                       # two calls in a row share the built-in buffer
            X, W = c.X.cuda(), c.W.cuda()
            ref = api.qf_fq_linear_fwd(X, W, wq, aq, y_dtype=torch.float32)
            Y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
            wts = torch.zeros(1, device="cuda") if wq == api.FMT_NVFP4 else None
            ats = torch.zeros(1, device="cuda") if aq == api.FMT_NVFP4 else None
            api.qf_fq_linear_fwd_noalloc(X, W, Y, wq, aq, w_tscale=wts, a_tscale=ats)
            torch.cuda.synchronize()
            # same kernels, same operands, same summation order: within the tolerance trivially, and in fact identical
            rms = ref.pow(2).mean().sqrt().item()
            assert (Y - ref).abs().max().item() <= TOL * rms
            assert torch.equal(Y, ref)
            # and against the oracle, like every other path
            y_ref = oracle.fq_linear_fwd(torch_to_bits(c.X), torch_to_bits(c.W), wq, aq)
            err = np.abs(Y.cpu().numpy().astype(np.float64) - y_ref).max()
            assert err <= TOL * np.sqrt(np.mean(np.square(y_ref.astype(np.float64))))
    # BF16 output through the same path
    X, W = c1.X.cuda(), c1.W.cuda()
    ref = api.qf_fq_linear_fwd(X, W, api.FMT_MXFP4, api.FMT_NONE)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    api.qf_fq_linear_fwd_noalloc(X, W, Y, api.FMT_MXFP4, api.FMT_NONE)
    assert torch.equal(Y, ref)


@pytest.mark.gpu
def test_noalloc_call_leaves_free_device_memory_unchanged():
    M, N, K = 512, 768, 1024
    c = synth.linear_case(M, N, K, seed=23, outlier_channels=1, device="cuda")
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    fmt = api.FMT_MXFP4
    api.qf_fq_linear_fwd_noalloc(c.X, c.W, Y, fmt, fmt)             # first call on this device: set-up happens here
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    reserved_before = torch.cuda.memory_reserved()
    for _ in range(3):
        api.qf_fq_linear_fwd_noalloc(c.X, c.W, Y, fmt, fmt)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before                                 # nothing was taken from (or returned to) the driver
    assert torch.cuda.memory_reserved() == reserved_before           # nor from torch's caching allocator
    # copies a previous caller left in the shared buffer are never trusted: the reuse flags are ignored
    c2 = synth.linear_case(M, N, K, seed=24, outlier_channels=1, device="cuda")
    Y2 = torch.empty_like(Y)
    api.qf_fq_linear_fwd_noalloc(c2.X, c2.W, Y2, fmt, fmt, flags=api.REUSE_W_HAT | api.REUSE_X_HAT)
    assert torch.equal(Y2, api.qf_fq_linear_fwd(c2.X, c2.W, fmt, fmt))


@pytest.mark.gpu
def test_noalloc_rejects_problems_beyond_the_built_in_buffer():
    # 4096 x 4096 weights alone fill 32 MiB: with the header and the activation copy it no longer fits
    M, N, K = 128, 4096, 4096
    X = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((N, K), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(api.QfError) as e:
        api.qf_fq_linear_fwd_noalloc(X, W, Y, api.FMT_MXFP4, api.FMT_MXFP4)
    assert e.value.code == 10
    assert "built-in buffer" in str(e.value)


def test_noalloc_size_check_needs_no_gpu():
    P = 0x10000
    f = api.lib().qf_fq_linear_fwd_noalloc
    assert f(P, P, P, 0, 1 << 40, 1 << 40, 1 << 40, 2, 2, None, None, 0, None) == 10
    assert f(P, P, P, 0, -1, 8, 32, 2, 2, None, None, 0, None) == 2
