"""GPU parity of the quantization-aware linear layer (forward and straight-through backward)
against the CPU oracle, through the C ABI. Tolerance (stated by the benchmark spec): max|diff| <= 1e-2 *
rms(reference), judged on FP32 outputs; BF16 outputs must be the BF16 rounding of the same
accumulator up to one unit in the last place."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39223_b200 import api, synth
from util import bits_to_f32, torch_to_bits

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _rms(a):
    return float(np.sqrt(np.mean(np.square(a.astype(np.float64)))))


def _close(got, ref, what):
    got = got.detach().float().cpu().numpy() if isinstance(got, torch.Tensor) else got
    err = float(np.abs(got.astype(np.float64) - ref.astype(np.float64)).max())
    bound = TOL * _rms(ref)
    assert err <= bound, f"{what}: max|diff| {err:.3e} > {bound:.3e}"


def _bf16_is_rounding_of(bf, f32, what):
    a = bf.float().cpu().numpy()
    b = f32.to(torch.bfloat16).float().cpu().numpy()
    ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(b), 1e-30))) - 7)
    assert np.all(np.abs(a - b) <= ulp * 1.0001), what


COMBOS = [(api.FMT_MXFP4, api.FMT_MXFP4), (api.FMT_NVFP4, api.FMT_NONE), (api.FMT_NVFP4, api.FMT_NVFP4),
          (api.FMT_Q4_K, api.FMT_NONE), (api.FMT_NONE, api.FMT_NONE), (api.FMT_MXFP4, api.FMT_NONE)]


@pytest.mark.parametrize("wq,aq", COMBOS)
@pytest.mark.parametrize("M,N,K", [(128, 256, 256), (200, 264, 768), (1, 8, 256), (333, 520, 1024)])
def test_small_complete_shapes(wq, aq, M, N, K):
    c = synth.linear_case(M, N, K, seed=M + N, outlier_channels=2)
    xb, wb, dyb = (torch_to_bits(t) for t in (c.X, c.W, c.dY))
    X, W, dY = c.X.cuda(), c.W.cuda(), c.dY.cuda()
    y_ref = oracle.fq_linear_fwd(xb, wb, wq, aq)
    dx_ref, dw_ref = oracle.fq_linear_bwd(dyb, xb, wb, wq, aq)
    y32 = api.qf_fq_linear_fwd(X, W, wq, aq, y_dtype=torch.float32)
    dx32, dw32 = api.qf_fq_linear_bwd(dY, X, W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32)
    _close(y32, y_ref, "Y")
    _close(dx32, dx_ref, "dX")
    _close(dw32, dw_ref, "dW")
    y16 = api.qf_fq_linear_fwd(X, W, wq, aq, y_dtype=torch.bfloat16)
    dx16, dw16 = api.qf_fq_linear_bwd(dY, X, W, wq, aq, dx_dtype=torch.bfloat16, dw_dtype=torch.bfloat16)
    _bf16_is_rounding_of(y16, y32, "Y bf16")
    _bf16_is_rounding_of(dx16, dx32, "dX bf16")
    _bf16_is_rounding_of(dw16, dw32, "dW bf16")


def _random_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        M = int(rng.choice([rng.integers(1, 128), rng.integers(128, 300), rng.integers(300, 900)]))
        N = 8 * int(rng.integers(1, 100))
        K = 32 * int(rng.integers(1, 48))
        out.append((M, N, K))
    return out


@pytest.mark.parametrize("M,N,K", _random_shapes(14, 2024))
def test_randomly_drawn_shapes(M, N, K):
    """Shapes drawn at random across the one-CTA / two-CTA dispatch boundary (256 rows), with ragged row, column
    and contraction tails in every combination, forward and both backward products, with and without quantizers."""
    c = synth.linear_case(M, N, K, seed=M * 7 + N + K, outlier_channels=1)
    xb, wb, dyb = (torch_to_bits(t) for t in (c.X, c.W, c.dY))
    X, W, dY = c.X.cuda(), c.W.cuda(), c.dY.cuda()
    for wq, aq in ((api.FMT_MXFP4, api.FMT_MXFP4), (api.FMT_NONE, api.FMT_NONE), (api.FMT_NVFP4, api.FMT_NVFP4)):
        y = api.qf_fq_linear_fwd(X, W, wq, aq, y_dtype=torch.float32)
        dx, dw = api.qf_fq_linear_bwd(dY, X, W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32)
        _close(y, oracle.fq_linear_fwd(xb, wb, wq, aq), f"Y {wq}/{aq}")
        dx_ref, dw_ref = oracle.fq_linear_bwd(dyb, xb, wb, wq, aq)
        _close(dx, dx_ref, f"dX {wq}/{aq}")
        _close(dw, dw_ref, f"dW {wq}/{aq}")


def test_one_hot_rows_read_out_quantized_weights_exactly():
    K, N = 256, 264
    W = synth.randn_bf16((N, K), 0.02, 1).cuda()
    eye = torch.eye(K, dtype=torch.bfloat16, device="cuda")
    y = api.qf_fq_linear_fwd(eye, W, api.FMT_NVFP4, api.FMT_NVFP4, y_dtype=torch.float32)
    w_hat = api.qf_qdq(api.FMT_NVFP4, W)["out"]
    assert torch.equal(y, w_hat.float().T)


def test_accumulate_dw_and_partial_requests():
    c = synth.linear_case(256, 256, 512, seed=3)
    X, W, dY = c.X.cuda(), c.W.cuda(), c.dY.cuda()
    dx, dw = api.qf_fq_linear_bwd(dY, X, W, api.FMT_MXFP4, api.FMT_MXFP4)
    acc = dw.clone()
    api.qf_fq_linear_bwd(dY, X, W, api.FMT_MXFP4, api.FMT_MXFP4, want_dx=False, dW=acc, flags=api.ACCUMULATE_DW)
    assert torch.allclose(acc, 2 * dw, rtol=1e-6, atol=0)
    dx2, none = api.qf_fq_linear_bwd(dY, None, W, api.FMT_MXFP4, api.FMT_MXFP4, want_dw=False)
    assert none is None and torch.equal(dx2, dx)


def test_status_word_is_clean_and_runs_are_deterministic():
    c = synth.linear_case(512, 512, 512, seed=4)
    X, W = c.X.cuda(), c.W.cuda()
    ws = api.workspace(api.OP_LINEAR_FWD, 512, 512, 512)
    a = api.qf_fq_linear_fwd(X, W, api.FMT_MXFP4, api.FMT_MXFP4, ws=ws)
    assert api.qf_read_status(ws) == 0
    b = api.qf_fq_linear_fwd(X, W, api.FMT_MXFP4, api.FMT_MXFP4, ws=ws)
    assert torch.equal(a, b)


def test_nvfp4_scales_written_back_and_amax_reported():
    c = synth.linear_case(256, 256, 256, seed=5)
    X, W = c.X.cuda(), c.W.cuda()
    wts = torch.zeros(1, device="cuda"); ats = torch.zeros(1, device="cuda"); amax = torch.zeros(1, device="cuda")
    api.qf_fq_linear_fwd(X, W, api.FMT_NVFP4, api.FMT_NVFP4, w_tscale=wts, a_tscale=ats, a_amax_out=amax)
    assert wts.item() == np.float32(oracle.qdq(api.FMT_NVFP4, torch_to_bits(c.W))["tensor_scale"])
    assert ats.item() == np.float32(oracle.qdq(api.FMT_NVFP4, torch_to_bits(c.X))["tensor_scale"])
    assert amax.item() == c.X.abs().max().item()
    # max|X| is reported whichever way the activations are handled (from the quantize pass where there is one)
    want = c.X.abs().max().item()
    running = torch.tensor([float(ats.item()) * 1.5], device="cuda")
    ws = api.workspace(api.OP_LINEAR_BWD, 256, 256, 256)
    y_ref = api.qf_fq_linear_fwd(X, W, api.FMT_MXFP4, api.FMT_MXFP4, y_dtype=torch.float32)
    for aq, flags, ats_in in ((api.FMT_NVFP4, api.A_TSCALE_GIVEN, running), (api.FMT_MXFP4, 0, None), (api.FMT_NONE, 0, None),
                              (api.FMT_MXFP4, api.FUSED_QDQ, None), (api.FMT_MXFP4, api.REUSE_X_HAT, None)):
        amax.fill_(-1.0)
        y = api.qf_fq_linear_fwd(X, W, api.FMT_MXFP4, aq, a_tscale=ats_in, a_amax_out=amax, flags=flags, ws=ws, y_dtype=torch.float32)
        assert amax.item() == want, (aq, flags)
        if aq == api.FMT_MXFP4:
            assert torch.equal(y, y_ref)                  # (the reuse case finds the previous iteration's copy of X_hat)
    # a supplied (tied / running) scale is honoured
    given = torch.tensor([float(wts.item()) * 2], device="cuda")
    y = api.qf_fq_linear_fwd(X, W, api.FMT_NVFP4, api.FMT_NONE, w_tscale=given, flags=api.W_TSCALE_GIVEN, y_dtype=torch.float32)
    ref = oracle.fq_linear_fwd(torch_to_bits(c.X), torch_to_bits(c.W), api.FMT_NVFP4, api.FMT_NONE, w_tscale=float(given.item()))
    _close(y, ref, "Y with given scale")


def test_full_size_mxfp4_linear_sampled_rows():
    """The benchmark's workload and launch configuration: X 8192x4096, W 12288x4096, dY 8192x12288,
    MXFP4 weights and activations. The oracle recomputes sampled output rows with full contractions."""
    M, N, K = 8192, 12288, 4096
    c = synth.linear_case(M, N, K, seed=0, device="cuda")
    ws = api.workspace(api.OP_LINEAR_BWD, M, N, K)
    y = api.qf_fq_linear_fwd(c.X, c.W, api.FMT_MXFP4, api.FMT_MXFP4, y_dtype=torch.float32, ws=ws)
    dx, dw = api.qf_fq_linear_bwd(c.dY, c.X, c.W, api.FMT_MXFP4, api.FMT_MXFP4, dx_dtype=torch.float32, dw_dtype=torch.float32, ws=ws)
    assert api.qf_read_status(ws) == 0
    rng = np.random.default_rng(0)
    rows = np.sort(rng.choice(M, 24, replace=False)); rows[0] = 0; rows[-1] = M - 1
    xb, wb = torch_to_bits(c.X), torch_to_bits(c.W)
    w_hat = oracle.qdq_out(api.FMT_MXFP4, wb)
    x_hat = oracle.qdq_out(api.FMT_MXFP4, xb)
    _close(y[rows], oracle.matmul_fwd(x_hat[rows], w_hat), "Y rows")
    dyb = torch_to_bits(c.dY)
    _close(dx[rows], oracle.matmul_dgrad(dyb[rows], w_hat), "dX rows")
    n_idx = np.sort(rng.choice(N, 16, replace=False)); n_idx[0] = 0; n_idx[-1] = N - 1
    _close(dw[n_idx], oracle.matmul_wgrad(dyb, x_hat, n_idx), "dW rows")


@pytest.mark.parametrize("y_dtype", [torch.float32, torch.bfloat16])
def test_output_with_more_than_2_to_the_31_elements(y_dtype):
    """A tall product whose output has 2.4e9 elements (and, in FP32, byte offsets past 2^33): sampled rows
    around the 2^31-element boundary and at both ends against the oracle, forward and dX."""
    M, N, K = 1048576, 2304, 64
    assert M * N > 2 ** 31
    X = synth.randn_bf16((M, K), 1.0, 31, device="cuda")
    W = synth.randn_bf16((N, K), 0.05, 32, device="cuda")
    fmt = api.FMT_MXFP4
    y = api.qf_fq_linear_fwd(X, W, fmt, fmt, y_dtype=y_dtype)
    boundary = 2 ** 31 // N
    rows = [0, 1, 255, 256, boundary - 1, boundary, boundary + 1, M - 257, M - 2, M - 1]
    xb, wb = torch_to_bits(X[rows].cpu()), torch_to_bits(W.cpu())
    ref = oracle.fq_linear_fwd(xb, wb, fmt, fmt)
    if y_dtype == torch.float32:
        _close(y[rows], ref, "Y rows")
    else:
        _bf16_is_rounding_of(y[rows], torch.from_numpy(ref), "Y rows (BF16)")
    assert bool((y != 0).any(dim=1).all())                       # no row was left unwritten
    del y
    # dX = dY . W_hat with the roles swapped: dY [M, N] is the large operand this time
    dY = synth.randn_bf16((M, N), 1e-3, 33, device="cuda")
    dx, _ = api.qf_fq_linear_bwd(dY, X, W, fmt, fmt, dx_dtype=torch.float32, want_dw=False)
    w_hat = oracle.qdq_out(fmt, wb)
    _close(dx[rows], oracle.matmul_dgrad(torch_to_bits(dY[rows].cpu()), w_hat), "dX rows")


def _grouped_reference(Xp, W, offs, wq, aq, dYp=None):
    G = W.shape[0]
    ys, dxs, dws = [], [], []
    for g in range(G):
        a, b = int(offs[g]), int(offs[g + 1])
        xb, wb = torch_to_bits(Xp[a:b]), torch_to_bits(W[g])
        if b > a:
            ys.append(oracle.fq_linear_fwd(xb, wb, wq, aq))
        if dYp is not None:
            dyb = torch_to_bits(dYp[a:b])
            if b > a:
                dx, dw = oracle.fq_linear_bwd(dyb, xb, wb, wq, aq)
            else:
                dx, dw = np.zeros((0, W.shape[2]), np.float32), np.zeros(W.shape[1:], np.float32)
            dxs.append(dx); dws.append(dw)
    return np.concatenate(ys), (np.concatenate(dxs) if dxs else None), (np.stack(dws) if dws else None)


@pytest.mark.parametrize("wq,aq", [(api.FMT_MXFP4, api.FMT_MXFP4), (api.FMT_NONE, api.FMT_NONE)])
def test_grouped_small_with_ragged_and_empty_experts(wq, aq):
    tokens, E, top_k, H, F = 96, 6, 2, 256, 264
    r = synth.moe_routing(tokens, E, top_k, seed=1)
    # force one empty expert by giving it no segment
    X = synth.randn_bf16((tokens, H), 1.0, 2)
    Xp = synth.gather_rows(X, r.token_of_row)
    W = synth.randn_bf16((E, F, H), 0.02, 3)
    dYp = synth.randn_bf16((Xp.shape[0], F), 1e-3, 4)
    dYp[r.token_of_row < 0] = 0
    offs = r.group_offsets
    y_ref, dx_ref, dw_ref = _grouped_reference(Xp, W, offs, wq, aq, dYp)
    offs_d = offs.cuda()
    y = api.qf_fq_grouped_linear_fwd(Xp.cuda(), W.cuda(), offs_d, wq, aq, y_dtype=torch.float32)
    dx, dw = api.qf_fq_grouped_linear_bwd(dYp.cuda(), Xp.cuda(), W.cuda(), offs_d, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32)
    _close(y, y_ref, "grouped Y")
    _close(dx, dx_ref, "grouped dX")
    _close(dw, dw_ref, "grouped dW")


@pytest.mark.parametrize("seed", range(8))
def test_grouped_randomly_drawn_segments(seed):
    """Expert counts, segment lengths (zero included; each padded to a multiple of 128 rows as the interface
    requires), widths and contraction lengths drawn at random: both grouped kernels (the two-CTA one and the
    one-CTA one it falls back to for short problems) against the per-expert oracle."""
    rng = np.random.default_rng(500 + seed)
    E = int(rng.integers(1, 12))
    blocks = rng.choice([0, 1, 1, 2, 3, 5], E)                      # 128-row blocks per expert
    if seed % 2 == 0:
        blocks[:] = np.minimum(blocks, 1)                            # short problems: fewer than 256 rows in total sometimes
    offs = torch.tensor(np.concatenate([[0], np.cumsum(blocks) * 128]), dtype=torch.int32)
    rows = int(offs[-1])
    if rows == 0:
        blocks[0] = 1; offs = torch.tensor(np.concatenate([[0], np.cumsum(blocks) * 128]), dtype=torch.int32); rows = int(offs[-1])
    F, H = 8 * int(rng.integers(1, 60)), 32 * int(rng.integers(1, 24))
    Xp = synth.randn_bf16((rows, H), 1.0, 10 + seed)
    real = torch.ones(rows, dtype=torch.bool)
    for g in range(E):                                               # the tail of each segment is padding: zero rows
        a, b = int(offs[g]), int(offs[g + 1])
        if b > a:
            real[b - int(rng.integers(0, 100)):b] = False
    Xp[~real] = 0
    W = synth.randn_bf16((E, F, H), 0.02, 20 + seed)
    dYp = synth.randn_bf16((rows, F), 1e-3, 30 + seed); dYp[~real] = 0
    for wq, aq in ((api.FMT_MXFP4, api.FMT_MXFP4), (api.FMT_NONE, api.FMT_NONE)):
        y_ref, dx_ref, dw_ref = _grouped_reference(Xp, W, offs, wq, aq, dYp)
        y = api.qf_fq_grouped_linear_fwd(Xp.cuda(), W.cuda(), offs.cuda(), wq, aq, y_dtype=torch.float32)
        dx, dw = api.qf_fq_grouped_linear_bwd(dYp.cuda(), Xp.cuda(), W.cuda(), offs.cuda(), wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32)
        _close(y, y_ref, "grouped Y")
        _close(dx, dx_ref, "grouped dX")
        _close(dw, dw_ref, "grouped dW")


@pytest.mark.parametrize("table", [[0, 256, 128, 512, 384, 768, 768], [0, 200, 64, 100000, -5, 700, 768], [768, 0, 0, 0, 0, 0, 0]])
def test_grouped_calls_force_a_malformed_segment_table_into_range(table):
    """The segment table is device memory the host cannot validate. The kernels force every entry to a multiple
    of 128 inside [0, rows], so a table that breaks the contract (not monotone, not aligned, out of range)
    yields numbers that mean nothing but finite ones, no error status, and a context that still works."""
    E, rows, F, H = 6, 768, 264, 256
    Xp = synth.randn_bf16((rows, H), 1.0, 61, device="cuda")
    W = synth.randn_bf16((E, F, H), 0.02, 62, device="cuda")
    dYp = synth.randn_bf16((rows, F), 1e-3, 63, device="cuda")
    offs = torch.tensor(table, dtype=torch.int32, device="cuda")
    fmt = api.FMT_MXFP4
    ws = api.workspace(api.OP_GROUPED_BWD, rows, F, H, E)
    y = api.qf_fq_grouped_linear_fwd(Xp, W, offs, fmt, fmt, y_dtype=torch.float32, ws=ws)
    dx, dw = api.qf_fq_grouped_linear_bwd(dYp, Xp, W, offs, fmt, fmt, dx_dtype=torch.float32, dw_dtype=torch.float32, ws=ws)
    torch.cuda.synchronize()
    assert api.qf_read_status(ws) == 0
    assert bool(torch.isfinite(dw).all())
    # a well-formed call right afterwards is correct
    good = torch.tensor([0, 128, 256, 384, 512, 640, 768], dtype=torch.int32)
    y_ref, _, _ = _grouped_reference(Xp.cpu(), W.cpu(), good, fmt, fmt)
    _close(api.qf_fq_grouped_linear_fwd(Xp, W, good.cuda(), fmt, fmt, y_dtype=torch.float32), y_ref, "Y after a bad table")


def test_grouped_empty_expert_gives_zero_dw():
    E, H, F = 3, 256, 256
    offs = torch.tensor([0, 128, 128, 256], dtype=torch.int32)        # expert 1 has no rows
    Xp = synth.randn_bf16((256, H), 1.0, 5)
    W = synth.randn_bf16((E, F, H), 0.02, 6)
    dYp = synth.randn_bf16((256, F), 1e-3, 7)
    y_ref, dx_ref, dw_ref = _grouped_reference(Xp, W, offs, api.FMT_MXFP4, api.FMT_MXFP4, dYp)
    dx, dw = api.qf_fq_grouped_linear_bwd(dYp.cuda(), Xp.cuda(), W.cuda(), offs.cuda(), api.FMT_MXFP4, api.FMT_MXFP4,
                                          dx_dtype=torch.float32, dw_dtype=torch.float32)
    assert torch.count_nonzero(dw[1]) == 0
    _close(dw, dw_ref, "grouped dW")
    _close(dx, dx_ref, "grouped dX")


def test_full_size_nvfp4_weight_only_32k_tokens_sampled_rows():
    """One 32K-token sequence through an up projection, NVFP4 weights, unquantized activations:
    X 32768x4096, W 14336x4096 (and the matching down-projection shape for the backward operands)."""
    M, N, K = 32768, 14336, 4096
    c = synth.linear_case(M, N, K, seed=4, device="cuda", outlier_channels=0)
    ws = api.workspace(api.OP_LINEAR_BWD, M, N, K)
    wts = torch.zeros(1, device="cuda")
    y = api.qf_fq_linear_fwd(c.X, c.W, api.FMT_NVFP4, api.FMT_NONE, y_dtype=torch.bfloat16, ws=ws, w_tscale=wts)
    dx, dw = api.qf_fq_linear_bwd(c.dY, c.X, c.W, api.FMT_NVFP4, api.FMT_NONE, dx_dtype=torch.bfloat16, dw_dtype=torch.float32, ws=ws)
    assert api.qf_read_status(ws) == 0
    rng = np.random.default_rng(4)
    rows = np.sort(rng.choice(M, 16, replace=False)); rows[0] = 0; rows[-1] = M - 1
    wb = torch_to_bits(c.W)
    qw = oracle.qdq(api.FMT_NVFP4, wb)
    assert wts.item() == np.float32(qw["tensor_scale"])
    w_hat = qw["out"]
    xb = torch_to_bits(c.X[torch.from_numpy(rows).cuda()])
    y_ref = oracle.matmul_fwd(xb, w_hat)
    # BF16 outputs: compare with the tolerance plus one BF16 rounding of the reference
    got = y[torch.from_numpy(rows).cuda()].float().cpu().numpy()
    assert np.all(np.abs(got - y_ref) <= TOL * _rms(y_ref) + np.abs(y_ref) * 2.0 ** -8)
    dyb = torch_to_bits(c.dY[torch.from_numpy(rows).cuda()])
    dx_ref = oracle.matmul_dgrad(dyb, w_hat)
    gdx = dx[torch.from_numpy(rows).cuda()].float().cpu().numpy()
    assert np.all(np.abs(gdx - dx_ref) <= TOL * _rms(dx_ref) + np.abs(dx_ref) * 2.0 ** -8)
    n_idx = np.sort(rng.choice(N, 8, replace=False)); n_idx[0] = 0; n_idx[-1] = N - 1
    dw_ref = oracle.matmul_wgrad(torch_to_bits(c.dY), torch_to_bits(c.X), n_idx)
    _close(dw[torch.from_numpy(n_idx).cuda()], dw_ref, "dW rows")


@pytest.mark.parametrize("shape", ["gate", "gate_up", "down"])
def test_full_size_moe_grouped_mxfp4_sampled_experts(shape):
    """128 experts, hidden 2048, expert MLP 768, 16384 tokens routed top-8: the gate projection
    (N=768, K=2048), gate and up as one weight (N=1536, the layout the benchmark times) and the down
    projection (N=2048, K=768), forward and backward over all 131072 routed rows; three experts checked in full."""
    tokens, E, top_k = 16384, 128, 8
    F, H = {"gate": (768, 2048), "gate_up": (1536, 2048), "down": (2048, 768)}[shape]      # F = N, H = K of this projection
    r = synth.moe_routing(tokens, E, top_k, seed=0)
    assert abs(int(r.counts.sum()) - tokens * top_k) == 0 and int(r.counts.min()) > 0
    X = synth.randn_bf16((tokens, H), 1.0, 1)
    Xp = synth.gather_rows(X, r.token_of_row).cuda()
    W = synth.randn_bf16((E, F, H), 0.02, 2, device="cuda")
    dYp = synth.randn_bf16((Xp.shape[0], F), 1e-3, 3, device="cuda")
    dYp[(r.token_of_row < 0).cuda()] = 0
    offs = r.group_offsets.cuda()
    fmt = api.FMT_MXFP4
    y = api.qf_fq_grouped_linear_fwd(Xp, W, offs, fmt, fmt, y_dtype=torch.float32)
    dx, dw = api.qf_fq_grouped_linear_bwd(dYp, Xp, W, offs, fmt, fmt, dx_dtype=torch.float32, dw_dtype=torch.float32)
    for g in (0, 57, 127):
        a, b = int(r.group_offsets[g]), int(r.group_offsets[g + 1])
        xb, wb, dyb = torch_to_bits(Xp[a:b]), torch_to_bits(W[g]), torch_to_bits(dYp[a:b])
        _close(y[a:b], oracle.fq_linear_fwd(xb, wb, fmt, fmt), f"expert {g} Y")
        dx_ref, dw_ref = oracle.fq_linear_bwd(dyb, xb, wb, fmt, fmt)
        _close(dx[a:b], dx_ref, f"expert {g} dX")
        _close(dw[g], dw_ref, f"expert {g} dW")


@pytest.mark.parametrize("wq,aq", [(api.FMT_MXFP4, api.FMT_MXFP4), (api.FMT_MXFP4, api.FMT_NONE), (api.FMT_NONE, api.FMT_MXFP4),
                                   (api.FMT_MXFP4, api.FMT_NVFP4)])
@pytest.mark.parametrize("M,N,K", [(256, 256, 256), (520, 776, 1024), (1024, 1024, 2048)])
def test_in_kernel_mxfp4_quantization_is_bitwise_the_workspace_path(wq, aq, M, N, K):
    """QF_FUSED_QDQ quantizes the staged shared-memory tiles inside the matmul kernel. The operands it
    produces are the same bits as the materialised copies, and the accumulation order is the same, so
    every output must be identical to the default path's, not merely close."""
    c = synth.linear_case(M, N, K, seed=M + K, outlier_channels=4)
    X, W, dY = c.X.cuda(), c.W.cuda(), c.dY.cuda()
    y0 = api.qf_fq_linear_fwd(X, W, wq, aq, y_dtype=torch.float32)
    dx0, dw0 = api.qf_fq_linear_bwd(dY, X, W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32)
    ws = api.workspace(api.OP_LINEAR_BWD, M, N, K)
    y1 = api.qf_fq_linear_fwd(X, W, wq, aq, y_dtype=torch.float32, flags=api.FUSED_QDQ, ws=ws)
    dx1, dw1 = api.qf_fq_linear_bwd(dY, X, W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32, flags=api.FUSED_QDQ, ws=ws)
    assert api.qf_read_status(ws) == 0
    assert torch.equal(y0, y1) and torch.equal(dx0, dx1) and torch.equal(dw0, dw1)
    # and against the oracle, like every other path
    _close(y1, oracle.fq_linear_fwd(torch_to_bits(c.X), torch_to_bits(c.W), wq, aq), "Y fused")


@pytest.mark.parametrize("wq,aq", [(api.FMT_MXFP4, api.FMT_MXFP4), (api.FMT_MXFP4, api.FMT_NONE)])
@pytest.mark.parametrize("M,N,K", [(200, 264, 768), (520, 776, 1024)])
def test_mxfp4_scale_rule_without_saturation_through_the_layer(wq, aq, M, N, K):
    """QF_MXFP4_NO_CLIP reaches both operands' quantizers, in the workspace path and in the in-kernel
    one (bitwise the same again), forward and backward, and matches the oracle under the same rule."""
    c = synth.linear_case(M, N, K, seed=3 * M + K, outlier_channels=4)
    X, W, dY = c.X.cuda(), c.W.cuda(), c.dY.cuda()
    xb, wb, dyb = torch_to_bits(c.X), torch_to_bits(c.W), torch_to_bits(c.dY)
    f = api.MXFP4_NO_CLIP
    y0 = api.qf_fq_linear_fwd(X, W, wq, aq, y_dtype=torch.float32, flags=f)
    dx0, dw0 = api.qf_fq_linear_bwd(dY, X, W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32, flags=f)
    _close(y0, oracle.fq_linear_fwd(xb, wb, wq, aq, mxfp4_noclip=True), "Y")
    dx_ref, dw_ref = oracle.fq_linear_bwd(dyb, xb, wb, wq, aq, mxfp4_noclip=True)
    _close(dx0, dx_ref, "dX")
    _close(dw0, dw_ref, "dW")
    # the rule matters: the default rule's output differs
    assert not torch.equal(y0, api.qf_fq_linear_fwd(X, W, wq, aq, y_dtype=torch.float32))
    ws = api.workspace(api.OP_LINEAR_BWD, M, N, K)
    y1 = api.qf_fq_linear_fwd(X, W, wq, aq, y_dtype=torch.float32, flags=f | api.FUSED_QDQ, ws=ws)
    dx1, dw1 = api.qf_fq_linear_bwd(dY, X, W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32, flags=f | api.FUSED_QDQ, ws=ws)
    assert api.qf_read_status(ws) == 0
    assert torch.equal(y0, y1) and torch.equal(dx0, dx1) and torch.equal(dw0, dw1)


def test_in_kernel_quantization_on_blocks_at_the_bottom_of_the_exponent_range():
    """The in-kernel transform rounds in packed BF16 arithmetic for ordinary blocks and falls back to the
    conversion route for all-zero blocks and blocks whose scale sits at either end of the exponent range.
    Operands that mix ordinary blocks with zero, subnormal and tiny ones must still give the default path's
    bits (compared as bit patterns), and finite results."""
    M, N, K = 512, 512, 1024
    rng = np.random.default_rng(77)
    def operand(rows):
        ng = rows * K // 32
        kind = rng.integers(0, 4, ng)                                   # 0 ordinary, 1 zero, 2 subnormal, 3 tiny normal
        e = np.where(kind == 0, rng.integers(110, 135, ng), np.where(kind == 2, 0, rng.integers(1, 12, ng)))
        bits = (rng.integers(0, 2, (ng, 32)) << 15) | ((e[:, None] + rng.integers(0, 3, (ng, 32))) << 7) | rng.integers(0, 128, (ng, 32))
        bits[kind == 1] &= 0x8000
        bits[kind == 2] &= 0x807F
        return torch.from_numpy(bits.astype(np.uint16).reshape(rows, K).view(np.int16)).view(torch.bfloat16).cuda()
    X, W = operand(M), operand(N)
    dY = synth.randn_bf16((M, N), 1e-3, 5, device="cuda")
    fmt = api.FMT_MXFP4
    y0 = api.qf_fq_linear_fwd(X, W, fmt, fmt, y_dtype=torch.float32)
    dx0, dw0 = api.qf_fq_linear_bwd(dY, X, W, fmt, fmt, dx_dtype=torch.float32, dw_dtype=torch.float32)
    ws = api.workspace(api.OP_LINEAR_BWD, M, N, K)
    y1 = api.qf_fq_linear_fwd(X, W, fmt, fmt, y_dtype=torch.float32, flags=api.FUSED_QDQ, ws=ws)
    dx1, dw1 = api.qf_fq_linear_bwd(dY, X, W, fmt, fmt, dx_dtype=torch.float32, dw_dtype=torch.float32, flags=api.FUSED_QDQ, ws=ws)
    assert api.qf_read_status(ws) == 0
    for a, b in ((y0, y1), (dx0, dx1), (dw0, dw1)):
        assert bool(torch.isfinite(a).all())
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    _close(y1, oracle.fq_linear_fwd(torch_to_bits(X.cpu()), torch_to_bits(W.cpu()), fmt, fmt), "Y")


@pytest.mark.parametrize("wq,aq", [(api.FMT_MXFP4, api.FMT_MXFP4), (api.FMT_NVFP4, api.FMT_NVFP4), (api.FMT_Q4_K, api.FMT_NONE)])
def test_a_whole_step_replays_from_a_cuda_graph(wq, aq):
    """Nothing in a call synchronises, allocates or reads device memory on the host, so forward and backward
    can be captured into a CUDA graph; replays with new input contents must equal the eager results bit for bit."""
    M, N, K = 512, 768, 1024
    c = synth.linear_case(M, N, K, seed=9, outlier_channels=2)
    X, W, dY = c.X.cuda(), c.W.cuda(), c.dY.cuda()
    ws = api.workspace(api.OP_LINEAR_BWD, M, N, K)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda"); dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((N, K), dtype=torch.float32, device="cuda")
    wts, ats = torch.zeros(1, device="cuda"), torch.zeros(1, device="cuda")

    def step():
        api.qf_fq_linear_fwd(X, W, wq, aq, ws=ws, Y=Y, w_tscale=wts, a_tscale=ats)
        api.qf_fq_linear_bwd(dY, X, W, wq, aq, ws=ws, dX=dX, dW=dW, w_tscale=wts, a_tscale=ats)
    step(); torch.cuda.synchronize()                       # first use outside capture (per-device kernel attributes)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    for seed in (1, 2):
        c2 = synth.linear_case(M, N, K, seed=100 + seed, outlier_channels=2)
        X.copy_(c2.X); W.copy_(c2.W); dY.copy_(c2.dY)
        g.replay(); torch.cuda.synchronize()
        got = (Y.clone(), dX.clone(), dW.clone())
        step(); torch.cuda.synchronize()
        assert torch.equal(got[0], Y) and torch.equal(got[1], dX) and torch.equal(got[2], dW)
        assert api.qf_read_status(ws) == 0


def test_independent_calls_on_two_streams():
    """Two layers, each with its own workspace, driven from two streams at once: the results are those of running
    them one after the other (the library keeps no state between calls)."""
    shapes = [(640, 512, 1024), (384, 1024, 512)]
    cases = [synth.linear_case(M, N, K, seed=40 + i, outlier_channels=1, device="cuda") for i, (M, N, K) in enumerate(shapes)]
    fmt = api.FMT_MXFP4
    serial = []
    for c, (M, N, K) in zip(cases, shapes):
        y = api.qf_fq_linear_fwd(c.X, c.W, fmt, fmt, y_dtype=torch.float32)
        dx, dw = api.qf_fq_linear_bwd(c.dY, c.X, c.W, fmt, fmt, dx_dtype=torch.float32, dw_dtype=torch.float32)
        serial.append((y, dx, dw))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    wss = [api.workspace(api.OP_LINEAR_BWD, *s) for s in shapes]
    for rep in range(5):
        outs = [None, None]
        for i in (0, 1):
            with torch.cuda.stream(streams[i]):
                c = cases[i]
                y = api.qf_fq_linear_fwd(c.X, c.W, fmt, fmt, y_dtype=torch.float32, ws=wss[i])
                dx, dw = api.qf_fq_linear_bwd(c.dY, c.X, c.W, fmt, fmt, dx_dtype=torch.float32, dw_dtype=torch.float32, ws=wss[i])
                outs[i] = (y, dx, dw)
        torch.cuda.synchronize()
        for i in (0, 1):
            assert all(torch.equal(a, b) for a, b in zip(outs[i], serial[i]))
            assert api.qf_read_status(wss[i]) == 0


def test_speculated_weight_scale_through_the_layer():
    """QF_W_TSCALE_SPECULATIVE in the linear calls: the weight's tensor scale carried from call to call as the next
    guess. First call (guess 0) misses, later ones hit, a changed weight misses again; outputs always equal the
    default path's bit for bit and w_tscale always ends up exact."""
    M, N, K = 384, 520, 1024
    c = synth.linear_case(M, N, K, seed=77, outlier_channels=2, device="cuda")
    wq, aq = api.FMT_NVFP4, api.FMT_NONE
    wts = torch.zeros(1, device="cuda")
    W = c.W.clone()
    for step in range(4):
        if step == 2:
            W[5, 7] = 3.0                                          # the weight changes: last step's scale is now wrong
        ref_ts = torch.zeros(1, device="cuda")
        y0 = api.qf_fq_linear_fwd(c.X, W, wq, aq, y_dtype=torch.float32, w_tscale=ref_ts)
        dx0, dw0 = api.qf_fq_linear_bwd(c.dY, c.X, W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32, w_tscale=ref_ts)
        y1 = api.qf_fq_linear_fwd(c.X, W, wq, aq, y_dtype=torch.float32, w_tscale=wts, flags=api.W_TSCALE_SPECULATIVE)
        dx1, dw1 = api.qf_fq_linear_bwd(c.dY, c.X, W, wq, aq, dx_dtype=torch.float32, dw_dtype=torch.float32, w_tscale=wts,
                                        flags=api.W_TSCALE_SPECULATIVE)
        assert wts.item() == ref_ts.item()
        assert torch.equal(y0, y1) and torch.equal(dx0, dx1) and torch.equal(dw0, dw1)


def test_bounded_wait_gives_up_and_reports_timeout():
    """A device-side wait that can never be satisfied must expire, report QF_ERR_TIMEOUT through the
    status word and leave the context usable (no trap, no hang)."""
    status, gave_up = api.qf_selftest_timeout(1 << 20)
    assert status == 7 and gave_up == 1
    assert "wait expired" in api.status_string(status)
    # the context still works
    x = synth.randn_bf16((4, 64), 1.0, 0, device="cuda")
    assert torch.equal(api.qf_qdq(api.FMT_MXFP4, x)["out"], api.qf_qdq(api.FMT_MXFP4, x)["out"])


@pytest.mark.parametrize("M,N,K", [(256, 8, 32), (257, 136, 96), (511, 264, 160), (127, 8, 32), (1, 16, 64), (640, 72, 4128)])
def test_edge_shapes_short_and_ragged_contractions(M, N, K):
    c = synth.linear_case(M, N, K, seed=K, outlier_channels=0)
    xb, wb, dyb = (torch_to_bits(t) for t in (c.X, c.W, c.dY))
    X, W, dY = c.X.cuda(), c.W.cuda(), c.dY.cuda()
    fmt = api.FMT_MXFP4
    _close(api.qf_fq_linear_fwd(X, W, fmt, fmt, y_dtype=torch.float32), oracle.fq_linear_fwd(xb, wb, fmt, fmt), "Y")
    dx, dw = api.qf_fq_linear_bwd(dY, X, W, fmt, fmt, dx_dtype=torch.float32, dw_dtype=torch.float32)
    dx_ref, dw_ref = oracle.fq_linear_bwd(dyb, xb, wb, fmt, fmt)
    _close(dx, dx_ref, "dX")
    _close(dw, dw_ref, "dW")


def test_bf16_gradient_accumulation_rounds_once():
    c = synth.linear_case(512, 256, 256, seed=9)
    X, W, dY = c.X.cuda(), c.W.cuda(), c.dY.cuda()
    _, dw32 = api.qf_fq_linear_bwd(dY, X, W, api.FMT_MXFP4, api.FMT_MXFP4, want_dx=False, dw_dtype=torch.float32)
    base = synth.randn_bf16((256, 256), 1e-2, 10, device="cuda")
    acc = base.clone()
    api.qf_fq_linear_bwd(dY, X, W, api.FMT_MXFP4, api.FMT_MXFP4, want_dx=False, dW=acc, flags=api.ACCUMULATE_DW)
    assert torch.equal(acc, (base.float() + dw32).to(torch.bfloat16))      # one rounding of the FP32 sum


def test_grouped_with_more_experts_than_the_pair_kernel_table_holds():
    E, H, F = 300, 256, 256                   # > 256 experts: served by the one-CTA kernel
    counts = torch.tensor([(i * 37) % 3 for i in range(E)])              # 0, 1 or 2 blocks of 128 rows
    offs = torch.zeros(E + 1, dtype=torch.int32); offs[1:] = torch.cumsum(counts * 128, 0)
    rows = int(offs[-1])
    Xp = synth.randn_bf16((rows, H), 1.0, 1); W = synth.randn_bf16((E, F, H), 0.02, 2); dYp = synth.randn_bf16((rows, F), 1e-3, 3)
    y_ref, dx_ref, dw_ref = _grouped_reference(Xp, W, offs, api.FMT_MXFP4, api.FMT_MXFP4, dYp)
    y = api.qf_fq_grouped_linear_fwd(Xp.cuda(), W.cuda(), offs.cuda(), api.FMT_MXFP4, api.FMT_MXFP4, y_dtype=torch.float32)
    dx, dw = api.qf_fq_grouped_linear_bwd(dYp.cuda(), Xp.cuda(), W.cuda(), offs.cuda(), api.FMT_MXFP4, api.FMT_MXFP4,
                                          dx_dtype=torch.float32, dw_dtype=torch.float32)
    _close(y, y_ref, "Y"); _close(dx, dx_ref, "dX"); _close(dw, dw_ref, "dW")


def test_grouped_odd_block_counts_on_the_pair_kernel():
    E, H, F = 7, 512, 264                     # segments of 1, 3, 0, 2, 5, 1, 4 blocks: odd ones end in half-used pair tiles
    counts = torch.tensor([1, 3, 0, 2, 5, 1, 4])
    offs = torch.zeros(E + 1, dtype=torch.int32); offs[1:] = torch.cumsum(counts * 128, 0)
    rows = int(offs[-1])
    Xp = synth.randn_bf16((rows, H), 1.0, 4); W = synth.randn_bf16((E, F, H), 0.02, 5); dYp = synth.randn_bf16((rows, F), 1e-3, 6)
    y_ref, dx_ref, dw_ref = _grouped_reference(Xp, W, offs, api.FMT_MXFP4, api.FMT_MXFP4, dYp)
    y = api.qf_fq_grouped_linear_fwd(Xp.cuda(), W.cuda(), offs.cuda(), api.FMT_MXFP4, api.FMT_MXFP4, y_dtype=torch.float32)
    dx, dw = api.qf_fq_grouped_linear_bwd(dYp.cuda(), Xp.cuda(), W.cuda(), offs.cuda(), api.FMT_MXFP4, api.FMT_MXFP4,
                                          dx_dtype=torch.float32, dw_dtype=torch.float32)
    _close(y, y_ref, "Y"); _close(dx, dx_ref, "dX"); _close(dw, dw_ref, "dW")
    assert torch.count_nonzero(dw[2]) == 0


def test_grouped_nvfp4_weights_have_one_tensor_scale_per_expert():
    E, H, F = 5, 256, 264
    counts = torch.tensor([2, 1, 0, 3, 1])
    offs = torch.zeros(E + 1, dtype=torch.int32); offs[1:] = torch.cumsum(counts * 128, 0)
    rows = int(offs[-1])
    Xp = synth.randn_bf16((rows, H), 1.0, 11)
    W = synth.randn_bf16((E, F, H), 0.02, 12)
    W = (W.float() * torch.tensor([1.0, 4.0, 0.25, 16.0, 0.5]).view(E, 1, 1)).to(torch.bfloat16)     # experts of different magnitude
    dYp = synth.randn_bf16((rows, F), 1e-3, 13)
    y_ref, dx_ref, dw_ref = _grouped_reference(Xp, W, offs, api.FMT_NVFP4, api.FMT_NONE, dYp)
    wts = torch.zeros(E, device="cuda")
    y = api.qf_fq_grouped_linear_fwd(Xp.cuda(), W.cuda(), offs.cuda(), api.FMT_NVFP4, api.FMT_NONE, y_dtype=torch.float32, w_tscale=wts)
    want = [np.float32(oracle.qdq(api.FMT_NVFP4, torch_to_bits(W[g]))["tensor_scale"]) for g in range(E)]
    assert [np.float32(v) for v in wts.cpu().tolist()] == want
    _close(y, y_ref, "Y")
    dx, dw = api.qf_fq_grouped_linear_bwd(dYp.cuda(), Xp.cuda(), W.cuda(), offs.cuda(), api.FMT_NVFP4, api.FMT_NONE,
                                          dx_dtype=torch.float32, dw_dtype=torch.float32, w_tscale=wts, flags=api.W_TSCALE_GIVEN)
    _close(dx, dx_ref, "dX"); _close(dw, dw_ref, "dW")
    with pytest.raises(api.QfError):          # the per-expert scale array is required
        api.qf_fq_grouped_linear_fwd(Xp.cuda(), W.cuda(), offs.cuda(), api.FMT_NVFP4, api.FMT_NONE)


def test_grouped_nvfp4_scales_are_final_before_any_block_is_quantized():
    """Experts large enough that many CTAs quantize each one: all of them must use the expert's finished tensor
    scale. Repeated, because a CTA that converted the shared word too early would only sometimes be caught."""
    E, H, F = 4, 1024, 1024
    offs = torch.tensor([0, 128, 256, 384, 512], dtype=torch.int32)
    Xp = torch.eye(128, H, dtype=torch.bfloat16).repeat(E, 1)                       # one-hot rows read out W_hat[:, :128]
    W = synth.randn_bf16((E, F, H), 0.02, 21)
    W = (W.float() * torch.tensor([1.0, 8.0, 0.125, 64.0]).view(E, 1, 1)).to(torch.bfloat16)
    want = [bits_to_f32(oracle.qdq_out(api.FMT_NVFP4, torch_to_bits(W[g])))[:, :128].T for g in range(E)]
    Xd, Wd, od = Xp.cuda(), W.cuda(), offs.cuda()
    for _ in range(10):
        wts = torch.zeros(E, device="cuda")
        y = api.qf_fq_grouped_linear_fwd(Xd, Wd, od, api.FMT_NVFP4, api.FMT_NONE, y_dtype=torch.float32, w_tscale=wts).cpu().numpy()
        for g in range(E):
            np.testing.assert_array_equal(y[g * 128:(g + 1) * 128], want[g])


@pytest.mark.parametrize("wq,aq", [(api.FMT_MXFP4, api.FMT_MXFP4), (api.FMT_NVFP4, api.FMT_NVFP4), (api.FMT_Q4_K, api.FMT_NONE)])
def test_backward_can_reuse_the_forwards_quantized_copies(wq, aq):
    M, N, K = 384, 520, 1024
    c = synth.linear_case(M, N, K, seed=31, outlier_channels=2)
    X, W, dY = c.X.cuda(), c.W.cuda(), c.dY.cuda()
    dx0, dw0 = api.qf_fq_linear_bwd(dY, X, W, wq, aq)                      # recomputes W_hat and X_hat (the default)
    ws = api.workspace(api.OP_LINEAR_BWD, M, N, K)
    wts = torch.zeros(1, device="cuda"); ats = torch.zeros(1, device="cuda")
    api.qf_fq_linear_fwd(X, W, wq, aq, ws=ws, w_tscale=wts, a_tscale=ats)
    dx1, dw1 = api.qf_fq_linear_bwd(dY, X, W, wq, aq, ws=ws, w_tscale=wts, a_tscale=ats,
                                    flags=api.REUSE_W_HAT | api.REUSE_X_HAT)
    assert torch.equal(dx0, dx1) and torch.equal(dw0, dw1)
