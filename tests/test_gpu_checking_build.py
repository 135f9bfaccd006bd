"""The checking build of the library (-DGS_DEBUG) stands in for a memory checker: every index
into a shared-memory table that the search kernels compute from table contents, and every
position the prologue writes a table entry to, is tested against its table first; a failed test
surfaces as GS_DEV_INTERNAL in the device status word (nothing traps).  This file re-runs the
parity tests that stress the tables hardest -- all configs, ragged sizes, the adversarial pools,
the largest tables, the stream of dependent rounds -- against that build: answers must still be
the oracle's and the status word must stay clean (each of those tests asserts a zero status)."""
import pytest

import workloads as W
import test_gpu_parity as T

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def checked():
    from paper_2605_16867_b200 import GoodServe
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    ctx = GoodServe(0, checking=True)
    yield ctx
    assert ctx.device_status() & 32 == 0          # GS_DEV_INTERNAL
    ctx.close()


def test_checking_build_reports_through_the_status_word(checked):
    """A clean run leaves the word at zero; the bit is part of the ABI's status enum."""
    from paper_2605_16867_b200 import DeviceStatus
    assert DeviceStatus.INTERNAL == 32
    T.run_config(checked, W.make_workload(0))
    assert checked.device_status() == 0


@pytest.mark.parametrize("cfg_id", [1, 2])
def test_configs_at_full_size(checked, cfg_id):
    T.run_config(checked, W.make_workload(cfg_id))


def test_largest_config(checked):
    T.run_config(checked, W.make_workload(3, n_active=3_000_001))


@pytest.mark.parametrize("M", [1, 3, 33, 127, 1023, 1024])
@pytest.mark.parametrize("N", [1, 33, 4099])
def test_ragged_sizes(checked, M, N):
    T.test_ragged_sizes(checked, M, N)


@pytest.mark.parametrize("case", range(len(T.FUZZ_CASES)))
def test_adversarial_pools(checked, case):
    T.test_pruned_search_is_exact_on_adversarial_pools(checked, case)


@pytest.mark.parametrize("case", range(len(T.RECORD_LIST_CASES)))
def test_record_lists_at_bucket_edges(checked, case):
    T.test_record_lists_at_bucket_edges_and_row_deadlines(checked, case)


@pytest.mark.parametrize("share,scarce_kv", [(1.0, False), (0.3, True), (0.01, True)])
def test_fallback_heavy_batches(checked, share, scarce_kv):
    T.test_fallback_heavy_and_sparse_batches(checked, share, scarce_kv)


def test_most_types_with_accumulate(checked):
    T.test_accumulate_with_the_most_types(checked)


def test_stream_of_dependent_rounds(checked):
    T.test_config4_stream(checked)


@pytest.mark.parametrize("case", [0, 4, 10])
def test_reroute_on_adversarial_pools(checked, case):
    T.test_reroute_on_adversarial_pools(checked, case)


@pytest.mark.parametrize("case", [3, 8])
def test_reroute_of_requests_that_are_not_at_risk(checked, case):
    T.test_reroute_of_requests_that_are_not_at_risk(checked, case)


@pytest.mark.parametrize("case", [4, 9])
def test_reroute_with_time_left_on_instance_estimates(checked, case):
    T.test_reroute_with_time_left_on_instance_estimates(checked, case)


@pytest.mark.parametrize("case", [0, 5, 13])
def test_prefix_on_adversarial_pools(checked, case):
    T.test_prefix_on_adversarial_pools(checked, case)


@pytest.mark.parametrize("case", [0, 3, 7])
def test_direct_on_adversarial_tables(checked, case):
    T.test_direct_on_adversarial_tables(checked, case)
