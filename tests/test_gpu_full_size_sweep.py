"""The scan-scaling sweep at its full size (B*T = 262144, H = 512, P = 256, bf16 I/O), in the
launch configuration bench.py times, against the float64 oracle on every output element."""
import numpy as np
import pytest

from paper_2502_20168_b200 import inputs as I
from tests.util import compare_layer, oracle_layer

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("w", I.C4, ids=[w.name for w in I.C4])
def test_sweep_point(w):
    from paper_2502_20168_b200 import harness
    d = I.draw_layer(w)
    res = harness.run_layer(d, w.io_dtype)
    ref = oracle_layer(d)
    errs = compare_layer(res, ref, w.io_dtype)
    print(w.name, {k: f"{v:.1e}" for k, v in errs.items()})
