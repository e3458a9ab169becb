"""Random sweep of small ragged workloads through the C interface against the fp64 oracle.

Shapes mix one-token prompts and branches, lengths either side of the 128-row tile edges, empty groups,
GQA ratios 1/2/4/7, both head dimensions, prompt-KV shards and lane counts from 1 to 148.  Every tensor
must meet the stated relative-L2 bound; every element must be within max(2e-2, six standard deviations of
its modelled rounding error) (`parity_util.rounding_error_sigma`): rows whose softmax sits on a handful of
keys carry bf16 roundings of dS that the flat 2e-2 does not cover, and this is where they are asserted
instead of avoided.
Three workloads in which an earlier sweep saw a 2.0e-2 .. 3.1e-2 element are listed by name.
"""
import numpy as np
import pytest
import torch

from paper_2609_33133_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

N_RANDOM = 45


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_33133_b200 import build
    build.build()
    from paper_2609_33133_b200 import binding
    return binding


def _random_case(case):
    rng = np.random.default_rng(9000 + case)
    ng = int(rng.integers(1, 4))
    pl = [int(rng.choice([1, 2, 17, 127, 128, 129, 255, 256, 257, 300, 511, 640, int(rng.integers(1, 900))])) for _ in range(ng)]
    bl = [[int(rng.choice([1, 2, 63, 127, 128, 129, 256, 257, int(rng.integers(1, 600))])) for _ in range(int(rng.integers(0, 5)))]
          for _ in range(ng)]
    hkv = int(rng.choice([1, 2, 4])); rep = int(rng.choice([1, 2, 4, 7])); d = int(rng.choice([64, 128]))
    splits = int(rng.choice([0, 0, 2, 3, 5])); lanes = int(rng.choice([0, 0, 1, 3, 7, 148]))
    return wl.Workload(f"sweep{case}", pl, bl, hkv * rep, hkv, d, 5000 + case), splits, lanes


# (prompt_len, branch_len, h_q, h_kv, d, shards, lanes, tensor seed): a 3.1e-2 / 2.4e-2 / 2.0e-2 element in dq_r / dq_p / dk_r
SEEN = {
    "one-token-prompts": ([1, 127, 1], [[129, 257, 2], [], []], 2, 1, 64, 0, 148, 5039),
    "tile-edge-prompts": ([128, 511, 255], [[128, 257, 1, 127], [129, 127, 128, 257], [129, 129, 1, 1]], 4, 4, 128, 0, 7, 5027),
    "two-token-prompt-g7": ([2, 255], [[63, 80], [257, 63]], 28, 4, 128, 2, 148, 5013),
}


def _check(B, w, splits, lanes, flags, handoff_limit=None):
    t = wl.make_tensors(w)
    got, _ = pu.run_gpu(B, w, t, kv_splits=splits, n_lanes=lanes, flags=flags, handoff_limit=handoff_limit)
    ref = pu.run_oracle(w, t)
    n_small = 2 * w.head_dim * w.h_q
    # a tensor of one or two rows: its relative-L2 figure is a couple of bf16 roundings, not a statistic
    # (same reasoning as the one-token case of test_gpu_parity); it keeps the element-wise bound
    tiny = {k for k in ref if ref[k].size and ref[k].size <= n_small}
    sigma = pu.rounding_error_sigma(w, t)
    rows = pu.errors(got, ref)
    pu.assert_parity_elementwise({k: v for k, v in got.items() if k not in tiny}, {k: v for k, v in ref.items() if k not in tiny}, sigma)
    for k in tiny:
        rel, mx, finite = rows[k]
        assert finite, k
        if k.startswith("lse"):
            assert mx <= pu.LSE_ABS, (k, mx)
        else:
            assert (np.abs(got[k] - ref[k]) <= np.maximum(pu.MAX_ABS, pu.SIGMAS * sigma[k])).all(), (k, mx)


@pytest.mark.parametrize("name", list(SEEN))
def test_workloads_that_exceeded_the_flat_bound(B, name):
    pl, bl, hq, hkv, d, splits, lanes, seed = SEEN[name]
    _check(B, wl.Workload(name, pl, bl, hq, hkv, d, seed), splits, lanes, 0)


@pytest.mark.parametrize("case", range(N_RANDOM))
def test_random_small_workloads(B, case):
    w, splits, lanes = _random_case(case)
    if w.total_response == 0 and splits:
        splits = 0
    _check(B, w, splits, lanes, B.FLAG_ZERO_PROMPT_GRAD if case % 2 else 0)


N_PADDED = 24


@pytest.mark.parametrize("case", range(N_PADDED))
def test_random_small_workloads_other_head_dims_and_handoff(B, case):
    """The same sweep recipe (its own seeds) over head dimensions that are padded to the 64- or 128-column tile, on
    the recomputing backward path (even cases) and on the dS hand-off path (odd cases)."""
    w, splits, lanes = _random_case(1000 + case)
    w.head_dim = int(np.random.default_rng(77 + case).choice([8, 16, 40, 56, 72, 80, 96, 104, 120]))
    if w.total_response == 0 and splits:
        splits = 0
    _check(B, w, splits, lanes, B.FLAG_ZERO_PROMPT_GRAD if case % 3 else 0, handoff_limit=(1 << 40) if case % 2 else 0)
