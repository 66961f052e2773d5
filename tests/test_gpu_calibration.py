"""The pipe-rate calibration launches behind the roofline denominators: they run, count their
instructions as documented and reject bad arguments. (Rates are reported by bench.py, not
asserted here: a shared GPU's clock is not a test condition.)"""
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def cp():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_13062_b200 import binding, build
    build.build()
    binding.lib()
    torch.cuda.set_device(0)
    return binding


def test_calibration_launches_count_and_order(cp):
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    threads = cp.CP_CALIBRATE_THREADS_PER_SM * sms
    seed = torch.linspace(0.5, 1.5, 10, device="cuda")
    sink = torch.full((threads,), float("nan"), device="cuda")
    rates = {}
    for kind, iters in ((0, 4000), (1, 4000), (2, 1000), (3, 4000), (4, 4000), (5, 4000), (6, 4000), (7, 4000)):
        n = cp.cp_calibrate_pipe(kind, seed, sink, iters)
        assert n == threads * iters * 8
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cp.cp_calibrate_pipe(kind, seed, sink, iters)
        e1.record()
        torch.cuda.synchronize()
        rates[kind] = n / (e0.elapsed_time(e1) * 1e-3)
        assert not torch.isnan(sink).any()       # every thread stored its result
    # the special-function pipe is the narrow one; the float pipe is at least as wide as the integer one
    assert rates[2] < rates[1] <= rates[0] * 1.05
    with pytest.raises(cp.CartpoleError):
        cp.cp_calibrate_pipe(8, seed, sink, 10)
    with pytest.raises(cp.CartpoleError):
        cp.cp_calibrate_pipe(0, seed, sink, 0)
