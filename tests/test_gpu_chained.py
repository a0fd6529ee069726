"""Two contractions launched back to back on one stream, the second reading what the first writes.
The short-K streaming kernel starts its set-up while the kernel before it in the stream still runs
(programmatic dependent launch); it must not read operand data before that kernel is complete."""
import numpy as np
import pytest
import torch

import helpers
import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    return helpers.api()


@pytest.fixture(scope="module")
def handle(api):
    return api.Handle()


def test_second_launch_sees_the_first_launch_s_result(api, handle):
    dtype = torch.float32
    m, k, n, q = 1024, 32, 64, 512
    A = helpers.random_tensor(9001, (m, k), None, dtype)
    B1 = helpers.random_tensor(9002, (k, n), None, dtype)
    B2 = helpers.random_tensor(9003, (n, q), None, dtype)
    D1 = helpers.random_tensor(9004, (m, n), None, dtype)
    D2 = helpers.random_tensor(9005, (m, q), None, dtype)
    dt = api.dtype_code(dtype)
    info = lambda t: api.TensorInfo(handle, dt, t.extents, t.strides)
    op1 = api.Contraction(handle, info(A), "mk", info(B1), "kn", None, "mn", info(D1), "mn", 1.0, 0.0)
    op2 = api.Contraction(handle, info(D1), "mn", info(B2), "nq", None, "mq", info(D2), "mq", 1.0, 0.0)
    for op in (op1, op2):
        op.set_attr(api.ATTR_KERNEL, api.KERNEL_TILED)
        op.set_attr(api.ATTR_VARIANT, 23)
        assert op.variant == 23
    dA, dB1, dB2, dD1, dD2 = (t.to("cuda") for t in (A, B1, B2, D1, D2))
    stream = torch.cuda.current_stream().cuda_stream
    ptr = lambda t: t.data_ptr()
    for rep in range(5):
        dD1.buffer.fill_(float("nan"))          # whatever the second launch reads too early is NaN
        dD2.buffer.fill_(0.0)
        op1.execute(stream, ptr(dA), ptr(dB1), 0, ptr(dD1))
        op2.execute(stream, ptr(dD1), ptr(dB2), 0, ptr(dD2))
        torch.cuda.synchronize()
        assert op1.device_error == 0 and op2.device_error == 0
        first = dD1.buffer.cpu()
        got = dD2.buffer.cpu()
        assert not torch.isnan(first).any() and not torch.isnan(got).any()
        # the oracle on what the first launch actually wrote
        X = D1.clone()
        X.buffer.copy_(first)
        want = D2.clone()
        scale = oracle.contract(X.numpy(), "mn", B2.numpy(), "nq", None, "mq", want.numpy(), "mq", 1.0, 0.0)
        pos = D2.offsets()
        assert helpers.compare(got[pos].numpy(), want.buffer[pos].numpy(), scale, dtype) <= 1.0
