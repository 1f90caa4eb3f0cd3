"""The bare FP8 UMMA stream the benchmark uses as the board's tensor ceiling: both forms run to completion with a
clean status word, and their rates are plausible and agree (a CTA pair does the same flops per SM)."""
import pytest
import torch

from paper_2607_11976_b200 import binding as lt

pytestmark = pytest.mark.gpu


def _rate(pair: bool, iters: int = 3000, launches: int = 10) -> float:
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    grid = n_sm & ~1 if pair else n_sm
    lt.lt_debug_umma_stream(pair, iters, status)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(launches):
        lt.lt_debug_umma_stream(pair, iters, status)
    e1.record()
    e1.synchronize()
    assert int(status.item()) == 0, "a bounded wait of the stream ran out"
    return grid * iters * 16777216.0 * launches / (e0.elapsed_time(e1) * 1e-3) / 1e12


def test_both_forms_run_and_agree():
    single = _rate(False)
    pair = _rate(True)
    # nominal dense FP8 peak is 4500 TFLOP/s; a stream that did not run, or ran a fraction of its UMMAs, is far off
    assert 1500.0 < single < 4600.0, single
    assert 1500.0 < pair < 4600.0, pair
    # the first measurement may still run at boost clocks and the second under the power limit (about 12 % apart);
    # a form that issued half or twice its UMMAs would be off by a factor of two
    assert abs(single - pair) / single < 0.35, (single, pair)


def test_bad_arguments_and_a_single_iteration():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(lt.LtError):
        lt.lt_debug_umma_stream(False, 0, status)
    with pytest.raises(lt.LtError):
        lt.lt_debug_umma_stream(True, (1 << 24) + 1, status)
    for pair in (False, True):
        for iters in (1, 2, 3):  # the two-deep commit ring with fewer iterations than slots
            lt.lt_debug_umma_stream(pair, iters, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
