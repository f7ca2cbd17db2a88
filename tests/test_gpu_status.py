"""The device-side error path: a bounded wait that nothing satisfies gives up, the kernel returns
normally, the host reads MX_ERR_TIMEOUT once, and the library keeps working afterwards."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mxb():
    from paper_2307_15517_b200 import binding
    return binding


def test_expired_wait_is_reported_and_cleared(mxb):
    assert mxb.mx_poll_status() == 0
    mxb.mx_selftest_wait_expiry(2000)                       # 2 ms
    assert mxb.mx_poll_status() == -7                       # MX_ERR_TIMEOUT
    assert mxb.mx_status_string(-7) == "device-side wait timed out"
    assert mxb.mx_poll_status() == 0                        # reading the status clears it
    # the context is intact: a product right after gives the right answer
    f = mxb.MxFormat(16, 4)
    x = torch.randn(256, 256, device="cuda")
    w = torch.randn(384, 256, device="cuda")
    wm, we = mxb.mx_quantize(w, f)
    y = mxb.mx_linear(x, f, wm, we, f, 384)
    y_simt = mxb.mx_linear(x, f, wm, we, f, 384, algo=mxb.MX_ALGO_SIMT)
    assert mxb.mx_poll_status() == 0
    assert np.allclose(y.cpu().numpy(), y_simt.cpu().numpy(), rtol=1e-5, atol=1e-5)
    with pytest.raises(mxb.MxError):
        mxb.mx_selftest_wait_expiry(0)
    with pytest.raises(mxb.MxError):
        mxb.mx_selftest_wait_expiry(10 ** 6)
