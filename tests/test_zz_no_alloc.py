"""The allocation-free projection entry point (`fdvlm_op_linear_static`) against the ordinary one.

Some hosts of this library may not call cudaMalloc at the point where they need a projection: they run under
another framework's allocator, under a fixed memory budget, or somewhere the implicit synchronisation of an
allocation is unwelcome.  For them the library carries its split-K scratch as a fixed device array.  This file
checks, through the C ABI, that the variant returns what `fdvlm_op_linear` returns -- on two calls in a row that
share (and overwrite) the same scratch -- and that a shape too large for the array is refused with a message.
Collected last on purpose (file name), so a failure here cannot hide the other tests' results."""
import pytest
import torch

from paper_2604_06832_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _case(m, n, k, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(m, k, generator=g)
    w = torch.randn(n, k, generator=g) * 0.05
    bias = torch.randn(n, generator=g) * 0.1
    if dtype == I.F32:
        return x.cuda(), w.cuda(), None, bias.cuda()
    if dtype == I.BF16:
        return x.to(torch.bfloat16).cuda(), w.to(torch.bfloat16).cuda(), None, bias.cuda()
    q, sc = I.quantize_e4m3_rows(w)
    return x.to(torch.bfloat16).cuda(), q.cuda(), sc.cuda(), bias.cuda()


@pytest.mark.parametrize("dtype", [I.BF16, I.F32, I.FP8])
def test_static_scratch_variant_matches_workspace_variant_twice_in_a_row(dtype):
    from paper_2604_06832_b200 import binding as B
    code = {I.F32: B.DT_F32, I.BF16: B.DT_BF16, I.FP8: B.DT_FP8}[dtype]
    # two different shapes back to back: the second call finds the first call's partial sums in the scratch
    shapes = [(32, 2560, 2048), (17, 1000, 1376)]
    for i, (m, n, k) in enumerate(shapes):
        x, w, sc, bias = _case(m, n, k, dtype, 100 + i)
        ref = B.op_linear(x, w, sc, bias, dtype=code)
        out = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda")
        B.op_linear_static(x, w, sc, bias, dtype=code, y=out)
        torch.cuda.synchronize()
        scale = max(float(ref.abs().max()), 1.0)
        err = float((out - ref).abs().max())
        assert err <= (2e-5 if dtype == I.F32 else 2e-4) * scale, (dtype, (m, n, k), err)
    # and the first shape once more, now after a different shape used the scratch
    m, n, k = shapes[0]
    x, w, sc, bias = _case(m, n, k, dtype, 100)
    assert torch.equal(B.op_linear_static(x, w, sc, bias, dtype=code), B.op_linear(x, w, sc, bias, dtype=code))


def test_static_scratch_variant_refuses_shapes_beyond_its_array():
    from paper_2604_06832_b200 import binding as B
    m, n, k = 64, 40000, 64          # 64 x 40000 fp32 outputs alone exceed 8 MiB of partial sums
    assert B.lib().fdvlm_op_linear_workspace_bytes(m, n, k, B.DT_BF16) > (8 << 20)
    x = torch.zeros(m, k, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(n, k, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.FdvlmError) as e:
        B.op_linear_static(x, w, dtype=B.DT_BF16)
    assert e.value.code == B.ERR_CAPACITY and "scratch" in str(e.value)
