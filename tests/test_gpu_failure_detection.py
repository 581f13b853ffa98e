"""Failure detection without a fault: the library's bounded barrier wait is made to run out on
a barrier that nothing completes (a short limit, a one-warp kernel of its own), the kernel
returns normally with PSA_DEVSTAT_WAIT_EXPIRED in the status word, the host helper maps the
word to PSA_ERR_TIMEOUT, and the same context then runs a correct psa_fwd."""
import pytest
import torch

from paper_2410_20305_b200 import binding as B
from paper_2410_20305_b200 import workloads as wl

from gpu_util import TOL_LSE, TOL_O, device_plan, max_abs, oracle_fwd, read_status

pytestmark = pytest.mark.gpu


def test_bounded_wait_expires_sets_status_and_context_stays_usable():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    limit = 2_000_000                      # about one millisecond of SM clock
    B.psa_selftest_wait_expiry(status, limit, waited)
    word = read_status(status)
    assert word & B.PSA_DEVSTAT_WAIT_EXPIRED
    assert B.psa_check_device_status(word) == 7          # PSA_ERR_TIMEOUT
    assert limit <= int(waited.item()) < 50 * limit      # it gave up at the limit, not far beyond
    # the context is intact: a forward pass right after is correct and reports nothing
    pack = wl.config_pack(0)
    q, k, v, _ = wl.attention_inputs(pack, 0)
    status.zero_()
    o, lse = B.psa_fwd(device_plan(pack), q.cuda(), k.cuda(), v.cuda(), status=status)
    assert read_status(status) == 0
    ro, rl = oracle_fwd(pack, q, k, v)
    assert max_abs(o, ro) <= TOL_O and max_abs(lse, rl) <= TOL_LSE
