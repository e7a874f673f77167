"""The L2 latency probe behind `report.py --topology`: every SM is covered once and the measured times are sane.  (Which
SMs end up on which side is a property of the individual GPU and is not asserted.)"""
import numpy as np
import pytest
import torch

from paper_2606_11718_b200 import binding as ccl

pytestmark = pytest.mark.gpu


def test_probe_covers_every_sm_once():
    nsm = torch.cuda.get_device_properties(0).multi_processor_count
    buf = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    lat, smid = ccl.ccl_probe_l2_latency(buf, 32, 4096, nsm)
    torch.cuda.synchronize()
    assert sorted(smid.cpu().tolist()) == list(range(nsm))             # one CTA per SM (they cannot share one)
    L = lat.cpu().numpy()
    assert np.isfinite(L).all() and L.min() > 50 and L.max() < 5000    # cycles per L2 round trip
    with pytest.raises(ValueError):
        ccl.ccl_probe_l2_latency(buf, 1024, 4096, nsm)                 # the lines would leave the buffer
    assert ccl.lib().ccl_probe_l2_latency(None, 1, 4096, 1, None, None, None) == ccl.ERR_INVALID_ARG
