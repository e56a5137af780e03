import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def golden_lines(name):
    """Yield the whitespace-split fields of every non-comment line of a golden text fixture."""
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if line:
                yield line.split()


@pytest.fixture(scope="session")
def fig1():
    """The paper's Fig. 1 layout and the values derived from it by hand."""
    g = dict(r_list={}, tokens=[], forced=[], free=[], seeded=[])
    for f in golden_lines("fig1_example.txt"):
        key = f[0]
        if key in ("nodes", "ranks_per_node", "slots_per_rank", "experts", "V_cobalt", "V_naive",
                   "coact_offdiag"):
            g[key] = int(f[1])
        elif key in ("slot_expert", "primary_slot", "replica_count", "nodes_mask", "load"):
            g[key] = [int(v) for v in f[1:]]
        elif key == "r_list":
            g["r_list"][(int(f[1]), int(f[2]))] = [int(v) for v in f[4:]]
        elif key == "token":
            g["tokens"].append(dict(t=int(f[1]), src=int(f[2]), ids=[int(f[3]), int(f[4])],
                                    cobalt=int(f[6]), naive=int(f[7])))
        elif key == "forced":
            g["forced"].append(tuple(int(v) for v in f[1:4]))
        elif key == "free":
            g["free"].append((int(f[1]), int(f[2]), [int(v) for v in f[4:]]))
        elif key == "seeded":
            g["seeded"].append(tuple(int(v) for v in f[1:5]))
        elif key == "ochiai_offdiag":
            g[key] = float(f[1])
        else:
            raise ValueError(f"unknown golden key {key}")
    return g
