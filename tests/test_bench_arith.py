"""Host arithmetic of bench.py that needs no GPU: which measured peak a roofline is divided by."""
import importlib.util
import os

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_roofline_peak_follows_the_sampled_clock():
    bench = _bench()
    peaks = {"bf16_burst": 1609.8, "bf16_sustained": 1365.0, "hbm": 6532.2, "source": "measured"}
    # stage loop at the boost clock: the burst cuBLAS figure, doubled for FP8
    peak, which, clock_peak, div = bench.roofline_peaks({"sm_mhz": 1965.0, "sm_max_mhz": 1965.0}, peaks, False, 148)
    assert (which, peak, div) == ("burst", 2 * 1609.8, 1.0)
    assert abs(clock_peak - 2 * 8192 * 148 * 1965e6 / 1e12) < 1e-9          # 4766 TFLOP/s
    # within 5 % of the maximum still counts as a burst; below it the sustained figure applies
    assert bench.roofline_peaks({"sm_mhz": 1870.0, "sm_max_mhz": 1965.0}, peaks, False, 148)[1] == "burst"
    peak, which, clock_peak, div = bench.roofline_peaks({"sm_mhz": 1785.0, "sm_max_mhz": 1965.0}, peaks, False, 148)
    assert (which, peak) == ("sustained", 2 * 1365.0)
    # BF16 mode: the BF16 figures themselves, half the FP8 rate per clock
    peak, which, clock_peak, div = bench.roofline_peaks({"sm_mhz": 1965.0, "sm_max_mhz": 1965.0}, peaks, True, 148)
    assert (which, peak, div) == ("burst", 1609.8, 2.0)
    assert abs(clock_peak - 8192 * 148 * 1965e6 / 1e12) < 1e-9
    # no clock sample: the cautious choice, and no clock-normalised figure
    peak, which, clock_peak, div = bench.roofline_peaks({}, peaks, False, 148)
    assert which == "sustained" and clock_peak is None


def test_bench_constants_match_the_stated_arithmetic():
    bench = _bench()
    assert bench.PRODUCTS == {"fwd": (1, 1), "bwd_delta": (1, 1), "bwd_dq": (2, 1), "bwd_dkdv": (2, 2)}
    assert sum(a + b for a, b in bench.PRODUCTS.values()) == 11               # executed products per pair
    assert bench.NOMINAL_FP8_TFLOPS == 4500.0 and bench.FP8_OVER_BF16 == 2.0
