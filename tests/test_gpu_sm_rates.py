"""kap_device_sm_rates: the per-SM streaming-rate measurement (a tool beside the path; nothing the
paper defines).  Checked for what must hold on any device: one positive rate per SM, mean 1, a
bounded spread, the cached second call returns the same numbers, and a too-small output array is
refused without being written."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2607_24260_b200 import kap

pytestmark = pytest.mark.gpu


def test_rates_are_positive_normalised_and_cached():
    n_sms = torch.cuda.get_device_properties(0).multi_processor_count
    r = kap.device_sm_rates(0)
    assert r.shape == (n_sms,) and r.dtype == np.float32
    assert np.all(r > 0.3) and np.all(r < 3.0)
    assert abs(float(r.mean()) - 1.0) < 1e-3
    np.testing.assert_array_equal(kap.device_sm_rates(0), r)


def test_small_output_array_is_refused():
    lib = kap.lib()
    out = np.full(4, -1.0, dtype=np.float32)
    n = C.c_int32(0)
    st = lib.kap_device_sm_rates(0, 4, out.ctypes.data_as(C.POINTER(C.c_float)), C.byref(n))
    assert st == kap.ERR_CAPACITY
    assert n.value == torch.cuda.get_device_properties(0).multi_processor_count
    assert np.all(out == -1.0)
