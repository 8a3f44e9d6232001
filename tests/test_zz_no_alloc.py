"""The allocation-free projection entry point (`fdvlm_op_linear_static`) against the ordinary one and the oracle.

Some hosts of this library may not call cudaMalloc at the point where they need a projection: they run under
another framework's allocator, under a fixed memory budget, or somewhere the implicit synchronisation of an
allocation is unwelcome.  For them the library carries its scratch as a fixed device array.  This file checks,
through the C ABI, that the variant returns what `fdvlm_op_linear` returns and what the plain definition gives -- on
calls in a row that share (and overwrite) the same scratch, the very first of them being the static one --, that the
device's free memory does not move across a call, that its status query reads clean, and that a shape too large for
the array is refused with a message.
Collected last on purpose (file name), so a failure here cannot hide the other tests' results."""
import numpy as np
import pytest
import torch

from oracle import fdvlm_oracle as orc
from paper_2604_06832_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _case(m, n, k, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(m, k, generator=g)
    w = torch.randn(n, k, generator=g) * 0.05
    bias = torch.randn(n, generator=g) * 0.1
    if dtype == I.F32:
        ref = x.double().numpy() @ w.double().numpy().T + bias.double().numpy()
        return x.cuda(), w.cuda(), None, bias.cuda(), ref
    xs = x.to(torch.bfloat16)
    xv = orc.to_f64(I.as_numpy_storage(xs))
    if dtype == I.BF16:
        ws = w.to(torch.bfloat16)
        ref = xv @ orc.to_f64(I.as_numpy_storage(ws)).T + bias.double().numpy()
        return xs.cuda(), ws.cuda(), None, bias.cuda(), ref
    q, sc = I.quantize_e4m3_rows(w)
    ref = xv @ (orc.to_f64(q.numpy()) * sc.double().numpy()[:, None]).T + bias.double().numpy()
    return xs.cuda(), q.cuda(), sc.cuda(), bias.cuda(), ref


@pytest.mark.parametrize("dtype", [I.BF16, I.F32, I.FP8])
def test_static_scratch_variant_matches_workspace_variant_and_oracle(dtype):
    from paper_2604_06832_b200 import binding as B
    code = {I.F32: B.DT_F32, I.BF16: B.DT_BF16, I.FP8: B.DT_FP8}[dtype]
    # two different shapes back to back: the second call finds the first call's partial sums in the scratch;
    # in each pair the static variant runs first, so in a fresh process it is the library's very first launch
    shapes = [(32, 2560, 2048), (17, 1000, 1376)]
    for i, (m, n, k) in enumerate(shapes):
        x, w, sc, bias, ref = _case(m, n, k, dtype, 100 + i)
        out = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda")
        B.op_linear_static(x, w, sc, bias, dtype=code, y=out)         # (its wrapper also reads the status query)
        torch.cuda.synchronize()
        scale = max(float(np.abs(ref).max()), 1.0)
        tol = (2e-5 if dtype == I.F32 else 2e-4) * scale
        assert float(np.abs(out.double().cpu().numpy() - ref).max()) <= tol, (dtype, (m, n, k))
        assert torch.equal(out, B.op_linear(x, w, sc, bias, dtype=code))
    # and the first shape once more, now after a different shape used the scratch
    m, n, k = shapes[0]
    x, w, sc, bias, _ = _case(m, n, k, dtype, 100)
    assert torch.equal(B.op_linear_static(x, w, sc, bias, dtype=code), B.op_linear(x, w, sc, bias, dtype=code))


def test_static_scratch_variant_allocates_no_device_memory():
    from paper_2604_06832_b200 import binding as B
    m, n, k = 32, 2048, 2048
    x, w, _, bias, _ = _case(m, n, k, I.BF16, 7)
    out = torch.empty(m, n, dtype=torch.float32, device="cuda")
    B.op_linear_static(x, w, None, bias, dtype=B.DT_BF16, y=out)      # first use on this device done
    torch.cuda.synchronize()
    for attempt in range(3):                                           # (another process on the GPU may move the figure)
        free0, _ = torch.cuda.mem_get_info()
        for _ in range(2):
            rc = B.lib().fdvlm_op_linear_static(x.data_ptr(), w.data_ptr(), None, bias.data_ptr(), out.data_ptr(), m, n, k,
                                                B.DT_BF16, None)
            assert rc == 0
        assert B.lib().fdvlm_op_linear_status(None, None) == 0
        free1, _ = torch.cuda.mem_get_info()
        if free0 == free1:
            break
    assert free0 == free1, (free0, free1)


def test_static_scratch_variant_refuses_shapes_beyond_its_array():
    from paper_2604_06832_b200 import binding as B
    m, n, k = 64, 40000, 64          # 64 x 40000 fp32 outputs alone exceed 8 MiB of partial sums
    assert B.lib().fdvlm_op_linear_workspace_bytes(m, n, k, B.DT_BF16) > (8 << 20)
    x = torch.zeros(m, k, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(n, k, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.FdvlmError) as e:
        B.op_linear_static(x, w, dtype=B.DT_BF16)
    assert e.value.code == B.ERR_CAPACITY and "scratch" in str(e.value)
