"""The one-kernel variant of the tensor-core path (state and apply pipelines side by side in every CTA).

The library picks the variant once per process from the environment (CASTLING_TC_ONE_KERNEL=1), so the cases
run in a child process.  Each case isolates one term of Eq. 9, as in test_gpu_term_isolation.py, on shapes
with several planes and many patches, for every packing of the tensor-core kernels and both filter sizes, and
checks that a single kernel was launched.
"""
from __future__ import annotations

import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, {root!r})
sys.path.insert(0, {root!r} + "/tests")
import workloads
from test_gpu_term_isolation import isolate, run_and_compare
# B, H, gridH, gridW, d, ksize, layout
cases = [(3, 5, 64, 64, 64, 3, "head_major"), (2, 3, 72, 80, 64, 5, "head_major"),
         (4, 6, 64, 64, 32, 3, "head_major"), (3, 4, 40, 132, 32, 5, "head_major"),
         (4, 6, 64, 64, 32, 3, "token_major"), (3, 4, 56, 72, 32, 5, "token_major"),
         (2, 8, 128, 128, 64, 3, "head_major")]
for B, H, gh, gw, d, ks, layout in cases:
    for term in ("conv", "linear", "halfsum"):
        c = workloads.custom_call(B, H, gh, gw, d, ks, "bf16", seed=7300 + B + H + gh + ks)
        run_and_compare(isolate(c, term), layout=layout, want_path=2, want_launches=1)
# the whole output on the largest sweep point's shape of one batch element less (8 planes of 256 x 256)
c = workloads.custom_call(1, 8, 256, 256, 64, 3, "bf16", seed=7399)
run_and_compare(c, want_path=2, want_launches=1)
print("one-kernel cases passed")
"""


def test_one_kernel_variant_in_a_child_process():
    env = dict(os.environ, CASTLING_TC_ONE_KERNEL="1")
    res = subprocess.run([sys.executable, "-c", CHILD.format(root=ROOT)], env=env, capture_output=True, text=True,
                         timeout=900)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "one-kernel cases passed" in res.stdout
