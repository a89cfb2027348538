"""The allocation-free forward entry point (for hosts that may not allocate device memory when they
call us: the scratch it needs is a fixed buffer inside the library) must give what the ordinary
entry point gives. Collected last on purpose; passes on its own and after the rest of the suite."""
import pytest
import torch

from paper_2609_39223_b200 import api, synth

TOL = 1e-2          # same bound as the other linear-layer tests: max|diff| <= 1e-2 * rms(reference)


def _check_same(got, ref):
    ref32, got32 = ref.float(), got.float()
    rms = ref32.pow(2).mean().sqrt().item()
    assert (got32 - ref32).abs().max().item() <= TOL * rms


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
            _check_same(Y, ref)
    # BF16 output through the same path
    X, W = c1.X.cuda(), c1.W.cuda()
    ref = api.qf_fq_linear_fwd(X, W, api.FMT_MXFP4, api.FMT_NONE)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    api.qf_fq_linear_fwd_noalloc(X, W, Y, api.FMT_MXFP4, api.FMT_NONE)
    _check_same(Y, ref)


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
