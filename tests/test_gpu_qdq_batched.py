"""GPU parity of the batched quantize-dequantize call: every tensor of a batch must come out exactly as the
oracle quantizes it on its own (codes, scales, tensor scale, dequantized values), whatever the mix of sizes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39223_b200 import api, synth
from util import torch_to_bits

pytestmark = pytest.mark.gpu
FMTS = [(api.FMT_NVFP4, "nvfp4"), (api.FMT_MXFP4, "mxfp4"), (api.FMT_Q4_K, "q4_k")]


def _tensors(shapes, seed, device="cuda"):
    out = []
    for i, (r, c) in enumerate(shapes):
        w = synth.weight_with_outliers(r, c, seed=seed + i, device=device) if r * c else torch.empty((r, c), dtype=torch.bfloat16, device=device)
        out.append((w.float() * (1.0 + 3.0 * (i % 5))).to(torch.bfloat16))         # tensors of different magnitude
    return out


def _check(fmt, b, xs, given=None):
    torch.cuda.synchronize()
    for i, x in enumerate(xs):
        ts = None if given is None else float(given[i])
        o = oracle.qdq(fmt, torch_to_bits(x), ts)
        np.testing.assert_array_equal(torch_to_bits(b.out[i]), o["out"], err_msg=f"tensor {i} out")
        np.testing.assert_array_equal(b.codes[i].cpu().numpy(), o["codes"], err_msg=f"tensor {i} codes")
        np.testing.assert_array_equal(b.scales[i].cpu().numpy(), o["scales"], err_msg=f"tensor {i} scales")
        if fmt == api.FMT_NVFP4:
            assert np.float32(b.tensor_scales[i].item()).tobytes() == np.float32(o["tensor_scale"]).tobytes(), f"tensor {i} scale"


MIXED = [(64, 1024), (1, 256), (300, 2304), (2048, 2048), (0, 512), (17, 256), (512, 4096), (129, 768)]


@pytest.mark.parametrize("fmt,name", FMTS)
def test_batch_of_mixed_sizes_equals_tensor_by_tensor(fmt, name):
    shapes = [(r, c - c % 256) for r, c in MIXED]
    xs = _tensors(shapes, 100)
    b = api.qf_qdq_batched(fmt, xs)
    _check(fmt, b, xs)
    # a second run over the same marshalled arguments (buffers hold the previous results) gives the same bits
    prev = [o.clone() for o in b.out]
    b.run()
    torch.cuda.synchronize()
    assert all(torch.equal(p, o) for p, o in zip(prev, b.out))


def test_nvfp4_batch_larger_than_l2_and_than_one_launch_table():
    """32 matrices of 2048 x 2048 (268 MB in: several L2-sized sub-batches) followed by 70 small ones (more than the
    64 tensors one launch carries): scales derived per tensor, a maximum never leaks into a neighbour."""
    xs = _tensors([(2048, 2048)] * 32 + [(8, 256)] * 70, 200)
    b = api.qf_qdq_batched(api.FMT_NVFP4, xs)
    torch.cuda.synchronize()
    scales = b.tensor_scales.cpu().numpy()
    for i, x in enumerate(xs):
        want = np.float32(x.abs().max().item()) / np.float32(2688.0)
        assert scales[i] == want, i
    for i in (0, 5, 31, 32, 95, 101):
        o = oracle.qdq(api.FMT_NVFP4, torch_to_bits(xs[i]))
        np.testing.assert_array_equal(torch_to_bits(b.out[i]), o["out"])
        np.testing.assert_array_equal(b.codes[i].cpu().numpy(), o["codes"])
        np.testing.assert_array_equal(b.scales[i].cpu().numpy(), o["scales"])


def test_nvfp4_batch_with_given_and_with_speculated_scales():
    shapes = [(256, 1024), (64, 512), (1024, 2048), (33, 256)]
    xs = _tensors(shapes, 300)
    derived = api.qf_qdq_batched(api.FMT_NVFP4, xs)
    torch.cuda.synchronize()
    # supplied scales (tied / running): 1.5x the derived ones
    given = (derived.tensor_scales * 1.5).contiguous()
    b = api.qf_qdq_batched(api.FMT_NVFP4, xs, tensor_scales=given.clone(), flags=api.TENSOR_SCALE_GIVEN)
    _check(api.FMT_NVFP4, b, xs, given=given.cpu().numpy())
    # speculated scales: zeros (all miss), the right ones (all hit), one wrong among right ones: always the derived result
    for guess in (torch.zeros(4, device="cuda"), derived.tensor_scales.clone(),
                  derived.tensor_scales * torch.tensor([1.0, 1.0, 2.0, 1.0], device="cuda")):
        b = api.qf_qdq_batched(api.FMT_NVFP4, xs, tensor_scales=guess.clone(), flags=api.TENSOR_SCALE_SPECULATIVE)
        _check(api.FMT_NVFP4, b, xs)


@pytest.mark.parametrize("fmt,name", FMTS)
def test_batch_in_place_and_partial_outputs(fmt, name):
    xs = _tensors([(128, 1024), (65, 512)], 400)
    ref = api.qf_qdq_batched(fmt, xs)
    torch.cuda.synchronize()
    only_codes = api.qf_qdq_batched(fmt, xs, want_out=False, want_scales=False)
    assert only_codes.out is None and all(torch.equal(a, b) for a, b in zip(only_codes.codes, ref.codes))
    # in place (out[i] = in[i]); with speculated scales the call must not let a first pass destroy its input
    work = [x.clone() for x in xs]
    b = api.QdqBatch(fmt, work, tensor_scales=torch.full((2,), 1e-3, device="cuda") if fmt == api.FMT_NVFP4 else None)
    b.out = work
    b._out = (api.c_void_p * 2)(*[t.data_ptr() for t in work])
    b.run(api.TENSOR_SCALE_SPECULATIVE if fmt == api.FMT_NVFP4 else 0)
    torch.cuda.synchronize()
    assert all(torch.equal(a, r) for a, r in zip(work, ref.out))
    assert all(torch.equal(a, r) for a, r in zip(b.codes, ref.codes))

