"""bench.py reports the DRAM traffic of committed ncu captures beside times it measures itself; the numbers in
bench.py must be the ones the profile summaries under profiles/ print (CPU only, no GPU run)."""
import importlib.util
import os
import re


def _bench(repo_root):
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(repo_root, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def _metric(text, name):
    """Value in bytes of a 'name  <number> <unit>' line of an ncu summary."""
    m = re.search(rf"^{re.escape(name)}\s+([0-9.]+)\s+(Gbyte|Mbyte|Kbyte|byte)", text, flags=re.M)
    assert m, name
    return float(m.group(1)) * {"Gbyte": 1e9, "Mbyte": 1e6, "Kbyte": 1e3, "byte": 1.0}[m.group(2)]


def _table_total(text, kernel):
    """read + write bytes of a kernel's row in the small-kernel table ('16 342 528 B  0 B')."""
    line = next(l for l in text.splitlines() if l.startswith(kernel))
    vals = re.findall(r"((?:\d{1,3} )*\d{1,3}) B", line)
    assert len(vals) == 2, line
    return sum(float(v.replace(" ", "")) for v in vals)


def test_traffic_constants_are_the_committed_profile_numbers(repo_root):
    bench = _bench(repo_root)
    for key, total in bench.NCU_TRAFFIC.items():
        terms = bench.NCU_TRAFFIC_SOURCE[key]
        assert abs(sum(v for *_, v in terms) - total) <= 1e-6 * total
        for fname, kernel, metric, value in terms:
            text = open(os.path.join(repo_root, "profiles", fname)).read()
            assert kernel in text, (fname, kernel)
            got = _table_total(text, kernel) if metric == "total" else _metric(text, metric)
            assert abs(got - value) <= 2e-3 * value, (fname, kernel, metric, got, value)
