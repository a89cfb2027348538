"""More GPU parity cases of the quantization-aware layer through the C ABI: the in-kernel quantizer over many
tiles per CTA pair, NVFP4 on both operands with supplied tensor scales, grouped layers with NVFP4 activations and
with Q4_K weights, and the down projection of the 32K-token workload at full size."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39223_b200 import api, synth
from util import torch_to_bits

pytestmark = pytest.mark.gpu
TOL = 1e-2          # max|diff| <= 1e-2 * rms(reference), on FP32 outputs


def _rms(a):
    return float(np.sqrt(np.mean(np.square(a.astype(np.float64)))))


def _close(got, ref, what):
    got = got.detach().float().cpu().numpy() if isinstance(got, torch.Tensor) else got
    err = float(np.abs(got.astype(np.float64) - ref.astype(np.float64)).max())
    bound = TOL * _rms(ref)
    assert err <= bound, f"{what}: max|diff| {err:.3e} > {bound:.3e}"


# (M, N, K): forward / dX / dW pair tiles and k-blocks per tile
#   2560 x 2304 x  832: 90 / 40 / 36 tiles, 13 / 36 / 40 k-blocks (13 is not a multiple of the 6-stage ring)
#   4096 x 8192 x  512: 512 / 32 / 64 tiles (seven per CTA pair in the forward), 8 / 128 / 64 k-blocks
#   1152 x 4608 x 1280: 90 / 25 / 90 tiles with a half-empty last row tile, 20 / 72 / 18 k-blocks
MULTI_TILE = [(2560, 2304, 832), (4096, 8192, 512), (1152, 4608, 1280)]


@pytest.mark.parametrize("wq,aq", [(api.FMT_MXFP4, api.FMT_MXFP4), (api.FMT_MXFP4, api.FMT_NONE), (api.FMT_NONE, api.FMT_MXFP4)])
@pytest.mark.parametrize("M,N,K", MULTI_TILE)
def test_in_kernel_quantization_over_many_tiles_per_cta_pair(wq, aq, M, N, K):
    """With more pair tiles than the 74 CTA pairs of the persistent grid, the in-kernel quantizer's running k-block
    counter, its stage and phase wrap across tiles, the transform groups running ahead of each other and the
    double-buffered accumulators are all exercised. Outputs must be the default path's bits, the status word clean,
    and sampled rows within tolerance of the oracle."""
    c = synth.linear_case(M, N, K, seed=M + N + K, outlier_channels=4, device="cuda")
    ws = api.workspace(api.OP_LINEAR_BWD, M, N, K)
    y0 = api.qf_fq_linear_fwd(c.X, c.W, wq, aq, y_dtype=torch.float32, ws=ws)
    dx0, dw0 = api.qf_fq_linear_bwd(c.dY, c.X, c.W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32, ws=ws)
    assert api.qf_read_status(ws) == 0
    y1 = api.qf_fq_linear_fwd(c.X, c.W, wq, aq, y_dtype=torch.float32, flags=api.FUSED_QDQ, ws=ws)
    dx1, dw1 = api.qf_fq_linear_bwd(c.dY, c.X, c.W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32,
                                    flags=api.FUSED_QDQ, ws=ws)
    assert api.qf_read_status(ws) == 0
    assert torch.equal(y0, y1), "Y"
    assert torch.equal(dx0, dx1), "dX"
    assert torch.equal(dw0, dw1), "dW"
    rng = np.random.default_rng(K)
    rows = np.sort(rng.choice(M, 12, replace=False)); rows[0] = 0; rows[-1] = M - 1
    n_idx = np.sort(rng.choice(N, 8, replace=False)); n_idx[0] = 0; n_idx[-1] = N - 1
    xb, wb, dyb = torch_to_bits(c.X), torch_to_bits(c.W), torch_to_bits(c.dY)
    w_hat, x_hat = oracle.qdq_out(wq, wb), oracle.qdq_out(aq, xb)
    _close(y1[rows], oracle.matmul_fwd(x_hat[rows], w_hat), "Y rows")
    _close(dx1[rows], oracle.matmul_dgrad(dyb[rows], w_hat), "dX rows")
    _close(dw1[n_idx], oracle.matmul_wgrad(dyb, x_hat, n_idx), "dW rows")


@pytest.mark.parametrize("M,N,K", [(200, 264, 768), (520, 776, 1024)])
def test_nvfp4_on_both_operands_with_supplied_tensor_scales(M, N, K):
    """NVFP4 weights and activations with both tensor scales handed in (a tied weight scale, a running activation
    scale): forward and backward against the oracle run with the same two scales, and the scale words left alone."""
    c = synth.linear_case(M, N, K, seed=N, outlier_channels=2)
    xb, wb, dyb = (torch_to_bits(t) for t in (c.X, c.W, c.dY))
    X, W, dY = c.X.cuda(), c.W.cuda(), c.dY.cuda()
    # scales a trainer could hold: 1.5x and 0.75x the ones the current tensors would derive (the second saturates blocks)
    for fw, fa in ((1.5, 1.5), (0.75, 2.0)):
        w_ts = np.float32(oracle.qdq(api.FMT_NVFP4, wb)["tensor_scale"]) * np.float32(fw)
        a_ts = np.float32(oracle.qdq(api.FMT_NVFP4, xb)["tensor_scale"]) * np.float32(fa)
        wts = torch.tensor([w_ts], dtype=torch.float32, device="cuda")
        ats = torch.tensor([a_ts], dtype=torch.float32, device="cuda")
        flags = api.W_TSCALE_GIVEN | api.A_TSCALE_GIVEN
        y = api.qf_fq_linear_fwd(X, W, api.FMT_NVFP4, api.FMT_NVFP4, y_dtype=torch.float32, w_tscale=wts, a_tscale=ats, flags=flags)
        dx, dw = api.qf_fq_linear_bwd(dY, X, W, api.FMT_NVFP4, api.FMT_NVFP4, dx_dtype=torch.float32, dw_dtype=torch.float32,
                                      w_tscale=wts, a_tscale=ats, flags=flags)
        assert wts.item() == w_ts and ats.item() == a_ts
        _close(y, oracle.fq_linear_fwd(xb, wb, api.FMT_NVFP4, api.FMT_NVFP4, w_tscale=float(w_ts), a_tscale=float(a_ts)), "Y")
        dx_ref, dw_ref = oracle.fq_linear_bwd(dyb, xb, wb, api.FMT_NVFP4, api.FMT_NVFP4, w_tscale=float(w_ts), a_tscale=float(a_ts))
        _close(dx, dx_ref, "dX")
        _close(dw, dw_ref, "dW")
        # the supplied scales matter: deriving them gives another result
        assert not torch.equal(y, api.qf_fq_linear_fwd(X, W, api.FMT_NVFP4, api.FMT_NVFP4, y_dtype=torch.float32))


def _segments(counts):
    offs = torch.zeros(len(counts) + 1, dtype=torch.int32)
    offs[1:] = torch.cumsum(torch.tensor(counts) * 128, 0)
    return offs


def _grouped_oracle(Xp, W, dYp, offs, wq, aq, w_ts=None, a_ts=None):
    ys, dxs, dws = [], [], []
    for g in range(W.shape[0]):
        a, b = int(offs[g]), int(offs[g + 1])
        wt = None if w_ts is None else float(w_ts[g])
        if b > a:
            xb, wb, dyb = torch_to_bits(Xp[a:b]), torch_to_bits(W[g]), torch_to_bits(dYp[a:b])
            ys.append(oracle.fq_linear_fwd(xb, wb, wq, aq, w_tscale=wt, a_tscale=a_ts))
            dx, dw = oracle.fq_linear_bwd(dyb, xb, wb, wq, aq, w_tscale=wt, a_tscale=a_ts)
        else:
            dx, dw = np.zeros((0, W.shape[2]), np.float32), np.zeros(tuple(W.shape[1:]), np.float32)
        dxs.append(dx); dws.append(dw)
    return np.concatenate(ys), np.concatenate(dxs), np.stack(dws)


def test_grouped_layer_with_nvfp4_activations_and_weights():
    """Grouped call, NVFP4 on both operands: one tensor scale per expert for the weights, a single activation scale
    for the whole routed input (derived here from all routed rows, then supplied in the backward)."""
    E, H, F = 5, 512, 264
    offs = _segments([2, 1, 0, 3, 2])
    rows = int(offs[-1])
    Xp = synth.randn_bf16((rows, H), 1.0, 41)
    W = synth.randn_bf16((E, F, H), 0.02, 42)
    W = (W.float() * torch.tensor([1.0, 4.0, 0.25, 8.0, 0.5]).view(E, 1, 1)).to(torch.bfloat16)
    dYp = synth.randn_bf16((rows, F), 1e-3, 43)
    a_ts = float(oracle.qdq(api.FMT_NVFP4, torch_to_bits(Xp))["tensor_scale"])          # over all routed rows
    w_ts = [np.float32(oracle.qdq(api.FMT_NVFP4, torch_to_bits(W[g]))["tensor_scale"]) for g in range(E)]
    y_ref, dx_ref, dw_ref = _grouped_oracle(Xp, W, dYp, offs, api.FMT_NVFP4, api.FMT_NVFP4, w_ts, a_ts)
    wts, ats = torch.zeros(E, device="cuda"), torch.zeros(1, device="cuda")
    y = api.qf_fq_grouped_linear_fwd(Xp.cuda(), W.cuda(), offs.cuda(), api.FMT_NVFP4, api.FMT_NVFP4, y_dtype=torch.float32,
                                     w_tscale=wts, a_tscale=ats)
    assert ats.item() == np.float32(a_ts) and [np.float32(v) for v in wts.cpu().tolist()] == w_ts
    _close(y, y_ref, "Y")
    dx, dw = api.qf_fq_grouped_linear_bwd(dYp.cuda(), Xp.cuda(), W.cuda(), offs.cuda(), api.FMT_NVFP4, api.FMT_NVFP4,
                                          dx_dtype=torch.float32, dw_dtype=torch.float32, w_tscale=wts, a_tscale=ats,
                                          flags=api.W_TSCALE_GIVEN | api.A_TSCALE_GIVEN)
    _close(dx, dx_ref, "dX")
    _close(dw, dw_ref, "dW")


def test_grouped_layer_with_q4k_weights():
    E, H, F = 4, 512, 264                 # K = 512: two super-blocks per weight row
    offs = _segments([1, 3, 0, 2])
    rows = int(offs[-1])
    Xp = synth.randn_bf16((rows, H), 1.0, 51)
    W = synth.randn_bf16((E, F, H), 0.02, 52)
    dYp = synth.randn_bf16((rows, F), 1e-3, 53)
    y_ref, dx_ref, dw_ref = _grouped_oracle(Xp, W, dYp, offs, api.FMT_Q4_K, api.FMT_NONE)
    y = api.qf_fq_grouped_linear_fwd(Xp.cuda(), W.cuda(), offs.cuda(), api.FMT_Q4_K, api.FMT_NONE, y_dtype=torch.float32)
    dx, dw = api.qf_fq_grouped_linear_bwd(dYp.cuda(), Xp.cuda(), W.cuda(), offs.cuda(), api.FMT_Q4_K, api.FMT_NONE,
                                          dx_dtype=torch.float32, dw_dtype=torch.float32)
    _close(y, y_ref, "Y"); _close(dx, dx_ref, "dX"); _close(dw, dw_ref, "dW")
    assert torch.count_nonzero(dw[2]) == 0


def test_full_size_nvfp4_weight_only_down_projection_sampled_rows():
    """The down projection of the 32K-token workload at full size: H 32768 x 14336, W_down 4096 x 14336, NVFP4
    weights, unquantized activations, forward and both backward products on sampled rows."""
    M, N, K = 32768, 4096, 14336
    c = synth.linear_case(M, N, K, seed=5, device="cuda", outlier_channels=0)
    ws = api.workspace(api.OP_LINEAR_BWD, M, N, K)
    wts = torch.zeros(1, device="cuda")
    y = api.qf_fq_linear_fwd(c.X, c.W, api.FMT_NVFP4, api.FMT_NONE, y_dtype=torch.float32, ws=ws, w_tscale=wts)
    dx, dw = api.qf_fq_linear_bwd(c.dY, c.X, c.W, api.FMT_NVFP4, api.FMT_NONE, dx_dtype=torch.float32, dw_dtype=torch.float32, ws=ws)
    assert api.qf_read_status(ws) == 0
    rng = np.random.default_rng(5)
    rows = np.sort(rng.choice(M, 12, replace=False)); rows[0] = 0; rows[-1] = M - 1
    sel = torch.from_numpy(rows).cuda()
    qw = oracle.qdq(api.FMT_NVFP4, torch_to_bits(c.W))
    assert wts.item() == np.float32(qw["tensor_scale"])
    _close(y[sel], oracle.matmul_fwd(torch_to_bits(c.X[sel]), qw["out"]), "Y rows")
    _close(dx[sel], oracle.matmul_dgrad(torch_to_bits(c.dY[sel]), qw["out"]), "dX rows")
    n_idx = np.sort(rng.choice(N, 4, replace=False)); n_idx[0] = 0; n_idx[-1] = N - 1
    dy_cols = torch_to_bits(c.dY[:, torch.from_numpy(n_idx).cuda()].contiguous())        # the 4 columns of dY those rows of dW need
    dw_ref = oracle.matmul_wgrad(dy_cols, torch_to_bits(c.X))
    _close(dw[torch.from_numpy(n_idx).cuda()], dw_ref, "dW rows")


def test_forward_with_an_empty_contraction_gives_zeros():
    X = torch.empty((300, 0), dtype=torch.bfloat16, device="cuda")
    W = torch.empty((264, 0), dtype=torch.bfloat16, device="cuda")
    for dt in (torch.float32, torch.bfloat16):
        Y = torch.full((300, 264), float("nan"), dtype=dt, device="cuda")
        api.qf_fq_linear_fwd(X, W, api.FMT_MXFP4, api.FMT_MXFP4, Y=Y)
        assert torch.count_nonzero(Y) == 0


@pytest.mark.parametrize("wq,aq", [(api.FMT_MXFP4, api.FMT_MXFP4), (api.FMT_MXFP4, api.FMT_NONE), (api.FMT_NONE, api.FMT_MXFP4)])
def test_in_kernel_quantization_in_grouped_layers(wq, aq):
    """QF_FUSED_QDQ in the per-expert calls: ragged, odd-length and empty segments, forward and both backward products,
    bit for bit the default path, and the default path against the per-expert oracle."""
    E, H, F = 7, 512, 520
    offs = _segments([1, 3, 0, 2, 5, 1, 4])
    rows = int(offs[-1])
    Xp = synth.randn_bf16((rows, H), 1.0, 61); W = synth.randn_bf16((E, F, H), 0.02, 62); dYp = synth.randn_bf16((rows, F), 1e-3, 63)
    Xd, Wd, dYd, od = Xp.cuda(), W.cuda(), dYp.cuda(), offs.cuda()
    ws = api.workspace(api.OP_GROUPED_BWD, rows, F, H, E)
    y0 = api.qf_fq_grouped_linear_fwd(Xd, Wd, od, wq, aq, y_dtype=torch.float32, ws=ws)
    dx0, dw0 = api.qf_fq_grouped_linear_bwd(dYd, Xd, Wd, od, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32, ws=ws)
    y1 = api.qf_fq_grouped_linear_fwd(Xd, Wd, od, wq, aq, y_dtype=torch.float32, ws=ws, flags=api.FUSED_QDQ)
    dx1, dw1 = api.qf_fq_grouped_linear_bwd(dYd, Xd, Wd, od, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32, ws=ws,
                                            flags=api.FUSED_QDQ)
    assert api.qf_read_status(ws) == 0
    assert torch.equal(y0, y1) and torch.equal(dx0, dx1) and torch.equal(dw0, dw1)
    y_ref, dx_ref, dw_ref = _grouped_oracle(Xp, W, dYp, offs, wq, aq)
    _close(y1, y_ref, "Y"); _close(dx1, dx_ref, "dX"); _close(dw1, dw_ref, "dW")


def test_in_kernel_quantization_full_size_moe_gate_up():
    """The 128-expert gate-and-up projection at full size with the quantizers inside the grouped matmul kernels."""
    tokens, E, top_k, F, H = 16384, 128, 8, 1536, 2048
    r = synth.moe_routing(tokens, E, top_k, seed=0)
    Xp = synth.gather_rows(synth.randn_bf16((tokens, H), 1.0, 1), r.token_of_row).cuda()
    W = synth.randn_bf16((E, F, H), 0.02, 2, device="cuda")
    dYp = synth.randn_bf16((Xp.shape[0], F), 1e-3, 3, device="cuda")
    dYp[(r.token_of_row < 0).cuda()] = 0
    offs = r.group_offsets.cuda()
    fmt = api.FMT_MXFP4
    ws = api.workspace(api.OP_GROUPED_BWD, Xp.shape[0], F, H, E)
    y0 = api.qf_fq_grouped_linear_fwd(Xp, W, offs, fmt, fmt, ws=ws)
    dx0, dw0 = api.qf_fq_grouped_linear_bwd(dYp, Xp, W, offs, fmt, fmt, ws=ws)
    y1 = api.qf_fq_grouped_linear_fwd(Xp, W, offs, fmt, fmt, ws=ws, flags=api.FUSED_QDQ)
    dx1, dw1 = api.qf_fq_grouped_linear_bwd(dYp, Xp, W, offs, fmt, fmt, ws=ws, flags=api.FUSED_QDQ)
    assert api.qf_read_status(ws) == 0
    assert torch.equal(y0, y1) and torch.equal(dx0, dx1) and torch.equal(dw0, dw1)


@pytest.mark.parametrize("wq,aq", [(api.FMT_NVFP4, api.FMT_NONE), (api.FMT_NVFP4, api.FMT_NVFP4), (api.FMT_MXFP4, api.FMT_NVFP4),
                                   (api.FMT_NVFP4, api.FMT_MXFP4)])
@pytest.mark.parametrize("M,N,K", [(520, 776, 1024), (2560, 2304, 832)])
@pytest.mark.parametrize("given", [False, True])
def test_in_kernel_nvfp4_quantization_is_bitwise_the_workspace_path(wq, aq, M, N, K, given):
    """QF_FUSED_QDQ with NVFP4 operands: the tensor scale is settled first (supplied, or derived by a maximum pass
    over the operand), then the matmul kernel quantizes the staged tiles with the stand-alone quantizer's arithmetic.
    Same bits as the default path, forward and backward; derived scales are written back all the same."""
    c = synth.linear_case(M, N, K, seed=M + K + 1, outlier_channels=3, device="cuda")
    ws = api.workspace(api.OP_LINEAR_BWD, M, N, K)
    def scales():
        if not given:
            return torch.zeros(1, device="cuda"), torch.zeros(1, device="cuda"), 0
        w_ts = np.float32(oracle.qdq(api.FMT_NVFP4, torch_to_bits(c.W))["tensor_scale"]) * np.float32(1.25)
        a_ts = np.float32(oracle.qdq(api.FMT_NVFP4, torch_to_bits(c.X))["tensor_scale"]) * np.float32(0.75)
        return (torch.tensor([w_ts], device="cuda"), torch.tensor([a_ts], device="cuda"), api.W_TSCALE_GIVEN | api.A_TSCALE_GIVEN)
    wts0, ats0, fl = scales()
    y0 = api.qf_fq_linear_fwd(c.X, c.W, wq, aq, y_dtype=torch.float32, ws=ws, w_tscale=wts0, a_tscale=ats0, flags=fl)
    dx0, dw0 = api.qf_fq_linear_bwd(c.dY, c.X, c.W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32, ws=ws,
                                    w_tscale=wts0, a_tscale=ats0, flags=fl)
    wts1, ats1, fl = scales()
    amax = torch.zeros(1, device="cuda")
    y1 = api.qf_fq_linear_fwd(c.X, c.W, wq, aq, y_dtype=torch.float32, ws=ws, w_tscale=wts1, a_tscale=ats1, a_amax_out=amax,
                              flags=fl | api.FUSED_QDQ)
    dx1, dw1 = api.qf_fq_linear_bwd(c.dY, c.X, c.W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32, ws=ws,
                                    w_tscale=wts1, a_tscale=ats1, flags=fl | api.FUSED_QDQ)
    assert api.qf_read_status(ws) == 0
    assert torch.equal(wts0, wts1) and torch.equal(ats0, ats1)
    assert amax.item() == c.X.abs().max().item()
    assert torch.equal(y0, y1), "Y"
    assert torch.equal(dx0, dx1), "dX"
    assert torch.equal(dw0, dw1), "dW"


def test_in_kernel_nvfp4_quantization_in_grouped_layers_with_per_expert_scales():
    E, H, F = 6, 512, 520
    offs = _segments([2, 3, 0, 1, 4, 2])
    rows = int(offs[-1])
    Xp = synth.randn_bf16((rows, H), 1.0, 71)
    W = synth.randn_bf16((E, F, H), 0.02, 72)
    W = (W.float() * torch.tensor([1.0, 4.0, 0.25, 8.0, 0.5, 2.0]).view(E, 1, 1)).to(torch.bfloat16)
    dYp = synth.randn_bf16((rows, F), 1e-3, 73)
    Xd, Wd, dYd, od = Xp.cuda(), W.cuda(), dYp.cuda(), offs.cuda()
    ws = api.workspace(api.OP_GROUPED_BWD, rows, F, H, E)
    out = []
    for fl in (0, api.FUSED_QDQ):
        wts, ats = torch.zeros(E, device="cuda"), torch.zeros(1, device="cuda")
        y = api.qf_fq_grouped_linear_fwd(Xd, Wd, od, api.FMT_NVFP4, api.FMT_NVFP4, y_dtype=torch.float32, ws=ws, w_tscale=wts,
                                         a_tscale=ats, flags=fl)
        dx, dw = api.qf_fq_grouped_linear_bwd(dYd, Xd, Wd, od, api.FMT_NVFP4, api.FMT_NVFP4, dx_dtype=torch.float32,
                                              dw_dtype=torch.float32, ws=ws, w_tscale=wts, a_tscale=ats, flags=fl)
        assert api.qf_read_status(ws) == 0
        out.append((y, dx, dw, wts, ats))
    for a, b in zip(*out):
        assert torch.equal(a, b)
    w_ts = [np.float32(oracle.qdq(api.FMT_NVFP4, torch_to_bits(W[g]))["tensor_scale"]) for g in range(E)]
    assert [np.float32(v) for v in out[1][3].cpu().tolist()] == w_ts
    a_ts = float(oracle.qdq(api.FMT_NVFP4, torch_to_bits(Xp))["tensor_scale"])
    y_ref, dx_ref, dw_ref = _grouped_oracle(Xp, W, dYp, offs, api.FMT_NVFP4, api.FMT_NVFP4, w_ts, a_ts)
    _close(out[1][0], y_ref, "Y"); _close(out[1][1], dx_ref, "dX"); _close(out[1][2], dw_ref, "dW")


@pytest.mark.parametrize("aq,given", [(api.FMT_MXFP4, False), (api.FMT_NVFP4, True)])
@pytest.mark.parametrize("M,N,K", [(520, 776, 1024), (2560, 2304, 832), (257, 264, 96)])
def test_backward_with_the_activation_pass_inside_the_dx_launch_is_bitwise_the_two_separate_products(aq, given, M, N, K):
    """A backward call that asks for both gradients lets spare warps of the dX launch quantize X for the dW product.
    The gradients must be the bits that two separate calls (dX alone, dW alone: no side job) produce."""
    c = synth.linear_case(M, N, K, seed=M + 3 * K, outlier_channels=2, device="cuda")
    wq = api.FMT_MXFP4
    ws = api.workspace(api.OP_LINEAR_BWD, M, N, K)
    ats = torch.tensor([0.01], device="cuda") if given else None
    fl = api.A_TSCALE_GIVEN if given else 0
    dx0, _ = api.qf_fq_linear_bwd(c.dY, c.X, c.W, wq, aq, dx_dtype=torch.float32, want_dw=False, ws=ws, a_tscale=ats, flags=fl)
    _, dw0 = api.qf_fq_linear_bwd(c.dY, c.X, c.W, wq, aq, dw_dtype=torch.float32, want_dx=False, ws=ws, a_tscale=ats, flags=fl)
    ws.zero_()                                    # nothing may be left over from the separate calls
    dx1, dw1 = api.qf_fq_linear_bwd(c.dY, c.X, c.W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32, ws=ws, a_tscale=ats, flags=fl)
    assert api.qf_read_status(ws) == 0
    assert torch.equal(dx0, dx1) and torch.equal(dw0, dw1)


def test_grouped_backward_with_the_activation_pass_inside_the_dx_launch():
    E, H, F = 7, 512, 520
    offs = _segments([1, 3, 0, 2, 5, 1, 4])
    rows = int(offs[-1])
    Xd = synth.randn_bf16((rows, H), 1.0, 81, device="cuda"); Wd = synth.randn_bf16((E, F, H), 0.02, 82, device="cuda")
    dYd = synth.randn_bf16((rows, F), 1e-3, 83, device="cuda"); od = offs.cuda()
    fmt = api.FMT_MXFP4
    ws = api.workspace(api.OP_GROUPED_BWD, rows, F, H, E)
    dx0, _ = api.qf_fq_grouped_linear_bwd(dYd, Xd, Wd, od, fmt, fmt, dx_dtype=torch.float32, want_dw=False, ws=ws)
    _, dw0 = api.qf_fq_grouped_linear_bwd(dYd, Xd, Wd, od, fmt, fmt, dw_dtype=torch.float32, want_dx=False, ws=ws)
    ws.zero_()
    dx1, dw1 = api.qf_fq_grouped_linear_bwd(dYd, Xd, Wd, od, fmt, fmt, dx_dtype=torch.float32, dw_dtype=torch.float32, ws=ws)
    assert api.qf_read_status(ws) == 0
    assert torch.equal(dx0, dx1) and torch.equal(dw0, dw1)


def test_weight_gradient_with_a_contraction_cut_into_chunks():
    """At 32768 tokens and more an FP32 dW is computed in chunks of 16384 tokens, the later launches adding into the
    first one's result. 40000 tokens give chunks of 16384 + 16384 + 7232 rows; with and without the caller's own
    accumulation flag, against the oracle."""
    M, N, K = 40000, 264, 96
    c = synth.linear_case(M, N, K, seed=77, outlier_channels=1)
    fmt = api.FMT_MXFP4
    _, dw_ref = oracle.fq_linear_bwd(torch_to_bits(c.dY), torch_to_bits(c.X), torch_to_bits(c.W), fmt, fmt)
    X, W, dY = c.X.cuda(), c.W.cuda(), c.dY.cuda()
    dw = torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda")
    api.qf_fq_linear_bwd(dY, X, W, fmt, fmt, want_dx=False, dW=dw)
    _close(dw, dw_ref, "dW")
    base = torch.randn((N, K), device="cuda") * 1e-2
    acc = base.clone()
    api.qf_fq_linear_bwd(dY, X, W, fmt, fmt, want_dx=False, dW=acc, flags=api.ACCUMULATE_DW)
    _close(acc - base, dw_ref, "dW accumulated")
    dw16 = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")           # BF16 output: one launch, no chunks
    api.qf_fq_linear_bwd(dY, X, W, fmt, fmt, want_dx=False, dW=dw16)
    assert (dw16.float() - dw).abs().max().item() <= dw.abs().max().item() * 2.0 ** -8
