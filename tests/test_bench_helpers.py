"""Host-side pieces of bench.py that need no GPU: the byte accounting of the roofline and the DRAM-traffic record."""
import importlib.util
import os

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_algorithmic_bytes_per_element(bench):
    """2 bytes read, 1 byte of code written, 2 bytes of scale and selection per block."""
    assert bench.alg_bytes((128, 128), 4096) == pytest.approx(3.0 + 2.0 / 16384)
    assert bench.alg_bytes((1, 128), 4096) == pytest.approx(3.0 + 2.0 / 128)


def test_traffic_record_belongs_to_the_current_kernel_sources(bench):
    """The DRAM counters under profiles/ are tied to a digest of the kernel sources; bench.py reports them only while
    the sources are the ones they were captured on.  A change under csrc/ without a new capture shows up here."""
    per_launch = bench.recorded_traffic(100663296)
    assert per_launch is not None, "profiles/main_kernel_blk128_keys_dram_traffic.txt was captured on other kernel sources"
    # every tile read once, every code written once: between 2.6 and 3.1 bytes per element reach DRAM
    assert 2.6 * 100663296 <= per_launch <= 3.1 * 100663296
