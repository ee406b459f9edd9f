"""A device wait that can never complete gives up within its limit and reports it (no hang, no trap)."""
import time

import pytest
import torch

from paper_2607_20457_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_wait_runs_out_and_reports_timeout_then_the_library_still_works():
    status = binding.new_status(DEV)
    result = torch.zeros(1, dtype=torch.int32, device=DEV)
    t0 = time.perf_counter()
    binding.wait_selftest(2_000_000, status, result)          # 2 ms limit
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 1.0
    assert int(status.item()) == binding.DEV_TIMEOUT
    assert int(result.item()) == 2                            # gave up, abort flag raised
    # the context is intact: a normal call afterwards succeeds
    pO = torch.randn(2, 8, 64, device=DEV)
    pL = torch.randn(2, 8, device=DEV)
    O, L = binding.pulsar_lse_merge(pO, pL)
    torch.cuda.synchronize()
    assert torch.isfinite(O.float()).all()


def test_limit_is_validated_on_the_host():
    with pytest.raises(binding.PulsarError):
        binding.wait_selftest(0, binding.new_status(DEV), torch.zeros(1, dtype=torch.int32, device=DEV))
    with pytest.raises(binding.PulsarError):
        binding.wait_selftest(5_000_000_000, binding.new_status(DEV), torch.zeros(1, dtype=torch.int32, device=DEV))
