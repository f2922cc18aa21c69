"""The cluster-per-plane variant of the tensor-core path (csrc/tc_cluster.cu): one thread-block cluster per (b,h)
plane builds the state in shares, adds the shares up through distributed shared memory and applies the sum, in
one launch without a workspace.

The library picks the variant once per process from the environment (CASTLING_TC_CLUSTER=1), so the cases run in
a child process.  Each case isolates one term of Eq. 9, as in test_gpu_term_isolation.py, for every packing of the
tensor-core kernels, both filter sizes, plane counts that lead to clusters of 8, 4 and 2 CTAs, a ragged last tile, and a plane so short that
some CTAs hold a single tile; every case must have taken exactly one launch.
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
# B, H, gridH, gridW, d, ksize, layout  (few planes take clusters of 8, more planes clusters of 4 or 2)
cases = [(2, 4, 64, 64, 64, 3, "head_major"),       # 8 planes
         (3, 5, 48, 64, 64, 5, "head_major"),       # 15 planes
         (2, 3, 40, 72, 64, 3, "head_major"),       # 6 planes, ragged last tile
         (4, 6, 64, 64, 32, 3, "head_major"),       # 24 planes of token pairs
         (8, 8, 64, 64, 32, 5, "head_major"),       # 64 planes of token pairs
         (4, 6, 64, 64, 32, 3, "token_major"),      # 12 planes of head pairs
         (2, 2, 24, 24, 64, 3, "head_major")]       # 4 planes of five tiles: some CTAs hold a single tile
for B, H, gh, gw, d, ks, layout in cases:
    for term in ("conv", "linear", "halfsum"):
        c = workloads.custom_call(B, H, gh, gw, d, ks, "bf16", seed=7500 + B + H + gh + ks)
        run_and_compare(isolate(c, term), layout=layout, want_path=2, want_launches=1)
# the whole output on a named configuration: the sweep point of 128 x 128 tokens
c = workloads.custom_call(2, 8, 128, 128, 64, 3, "bf16", seed=7599)
run_and_compare(c, want_path=2, want_launches=1)
print("cluster cases passed")
"""


def test_cluster_variant_in_a_child_process():
    env = dict(os.environ, CASTLING_TC_CLUSTER="1")
    res = subprocess.run([sys.executable, "-c", CHILD.format(root=ROOT)], env=env, capture_output=True, text=True,
                         timeout=900)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "cluster cases passed" in res.stdout
