"""Philox words, three ways, integer-exact: the CPU oracle, the library's device function and
cuRAND's header-only device function, over random counters and keys (all six words varied);
and the device Gumbel transform against the oracle's."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import santapp_oracle as orc
from tests.cuda import build_philox_check

pytestmark = pytest.mark.gpu


def test_device_philox_matches_curand_and_oracle():
    lib = ctypes.CDLL(build_philox_check.build())
    lib.philox_check_run.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                     ctypes.c_void_p]
    rng = np.random.default_rng(5)
    n = 4096
    ck = rng.integers(0, 1 << 32, size=(n, 6), dtype=np.uint64).astype(np.uint32)
    ck[0] = 0
    ck[1] = 0xFFFFFFFF
    ck[2] = [0, 1, 2, 3, 4, 5]
    d_ck = torch.from_numpy(ck.view(np.int32)).cuda()
    mine = torch.zeros((n, 4), dtype=torch.int32, device="cuda")
    theirs = torch.zeros((n, 4), dtype=torch.int32, device="cuda")
    gum = torch.zeros((n, 4), dtype=torch.float64, device="cuda")
    assert lib.philox_check_run(d_ck.data_ptr(), n, mine.data_ptr(), theirs.data_ptr(), gum.data_ptr()) == 0
    mine = mine.cpu().numpy().view(np.uint32)
    theirs = theirs.cpu().numpy().view(np.uint32)
    gum = gum.cpu().numpy()
    assert np.array_equal(mine, theirs)
    for i in range(0, n, 7):
        o = orc.philox4x32_10(ck[i, :4], ck[i, 4:])
        assert np.array_equal(o, mine[i])
        for w in range(4):
            g = orc.gumbel(int(o[w]))
            assert abs(gum[i, w] - g) <= 4e-15 * max(1.0, abs(g))
