import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the sm_100a kernels)")


def load_golden(name):
    """Parses a hand-written fixture under tests/golden/: 'key: hex words' lines and a 'stream:' hex block."""
    import numpy as np

    fields, stream, in_stream = {}, [], False
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            if in_stream:
                stream += [int(b, 16) for b in line.split()]
            elif line == "stream:":
                in_stream = True
            else:
                k, v = line.split(":", 1)
                fields[k.strip()] = v.split()
    out = {
        "nbits": int(fields["nbits"][0]),
        "cur": np.array([int(w, 16) for w in fields["cur_bits"]], np.uint32).view(np.float32),
        "recovered": np.array([int(w, 16) for w in fields["recovered_bits"]], np.uint32).view(np.float32),
        "stream": np.array(stream, np.uint8),
    }
    return out


@pytest.fixture(scope="session")
def oracle():
    from oracle import lc_oracle

    lc_oracle.lib()
    return lc_oracle
