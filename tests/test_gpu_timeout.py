"""The error path of the bounded device-side waits, exercised without a fault: a wait that
nothing satisfies gives up by itself, the status is reported once, the device stays usable."""
import numpy as np
import pytest
import torch

import paper_1603_05279_b200 as X
from paper_1603_05279_b200 import binding as B
from util import dev, host

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_once_and_the_device_stays_usable(oracle):
    X.xnor_check_device()                       # clean to begin with
    X.xnor_selftest_wait_timeout()
    with pytest.raises(X.XnorError) as e:
        X.xnor_check_device()
    assert e.value.status == B.XNOR_ERR_TIMEOUT
    X.xnor_check_device()                       # the word was cleared by the report
    # and an ordinary block still runs and is right
    g = np.random.Generator(np.random.Philox(77))
    x = g.standard_normal((2, 64, 9, 9)).astype(np.float32)
    w = g.standard_normal((48, 64, 3, 3)).astype(np.float32)
    d = B.xnor_conv_desc(2, 64, 9, 9, 48, 3, 3, 1, 1)
    wp, alpha = X.alloc_weights(48, 64, 3, 3)
    xp, A, K = X.alloc_binactiv(d)
    out = X.alloc_out(d)
    acc = X.alloc_out(d, torch.int32)
    X.xnor_binarize_weights(dev(w), wp, alpha)
    X.xnor_binactiv(dev(x), None, None, d, xp, A, K)
    X.xnor_conv2d_forward(xp, wp, alpha, K, None, d, out, acc)
    X.xnor_check_device()
    r = oracle.xnor_block(x, w, 1, 1)
    assert np.array_equal(host(acc), r.acc)
