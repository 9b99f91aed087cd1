"""Trace kernel vs oracle, bit for bit."""
import numpy as np
import pytest
import torch

from paper_2508_13231_b200 import workloads as wl
from gpu_util import to_np, trace_on_gpu

pytestmark = pytest.mark.gpu
Q16 = 65536


@pytest.fixture(scope="module")
def kvp():
    from paper_2508_13231_b200 import kvp
    return kvp


@pytest.mark.parametrize("name", ["tiny", "single_head", "layer_8b"])
def test_trace_named_configs_full(kvp, oracle, name):
    tp = wl.trace_params(name, seed=0)
    want = oracle.trace_generate(**tp)
    assert np.array_equal(to_np(trace_on_gpu(kvp, tp)), want)
    assert np.array_equal(to_np(trace_on_gpu(kvp, tp, kvp.TRACE_SINGLE_PASS)), want)


@pytest.mark.parametrize("name,groups", [("full_8b", [0, 101, 255]), ("long_70b", [0, 317, 639])])
def test_trace_full_size_sampled_groups(kvp, oracle, name, groups):
    # the full-size trace on the GPU; the oracle recomputes sampled (layer, head) groups, which are independent
    tp = wl.trace_params(name, seed=0)
    got = to_np(trace_on_gpu(kvp, tp))
    n, k, S = tp["units_per_group"], tp["topk"], tp["steps"]
    w = n // 32
    for g in groups:
        want = oracle.trace_generate(**tp, group_begin=g, group_count=1)
        assert np.array_equal(got[:, g * w:(g + 1) * w], want[:, g * w:(g + 1) * w]), g
    # property at full size: exactly k bits per group and step
    pop = np.unpackbits(got.view(np.uint8), axis=1).reshape(S, tp["groups"], n).sum(axis=2)
    assert np.all(pop == k)


@pytest.mark.parametrize("G,n,S,k", [(3, 40, 12, 7), (1, 16, 5, 16), (5, 100, 9, 1), (2, 1024, 6, 100),
                                     (2, 2048 + 64, 4, 33), (1, 8192, 3, 500), (7, 33, 40, 5),
                                     (151, 1030, 3, 70)])  # enough units for the score kernel with a thread per unit
@pytest.mark.parametrize("flags", [0, 1])          # two passes over a score matrix / single fused pass
def test_trace_ragged_shapes(kvp, oracle, G, n, S, k, flags):
    rng = np.random.default_rng(G * 1000 + n)
    base = (rng.integers(-3 * Q16, 3 * Q16, size=G * n)).astype(np.int32)
    tp = dict(groups=G, units_per_group=n, steps=S, topk=k, seed=77, rho_q=int(0.9 * Q16), c_q=int(0.4 * Q16),
              sigma_q=Q16, burst_jump=3 * Q16, burst_thr=int(0.05 * 2 ** 32), base=base)
    assert np.array_equal(to_np(trace_on_gpu(kvp, tp, flags)), oracle.trace_generate(**tp))


def test_trace_ties_go_to_lower_index(kvp, oracle):
    # no noise: scores are the coarse `base`, full of ties inside and across warps
    G, n, S, k = 2, 4096, 3, 1000
    rng = np.random.default_rng(5)
    base = (rng.integers(0, 4, size=G * n) * 1000).astype(np.int32)
    tp = dict(groups=G, units_per_group=n, steps=S, topk=k, seed=1, rho_q=Q16, c_q=0, sigma_q=0, burst_jump=0,
              burst_thr=0, base=base)
    assert np.array_equal(to_np(trace_on_gpu(kvp, tp)), oracle.trace_generate(**tp))
    assert np.array_equal(to_np(trace_on_gpu(kvp, tp, kvp.TRACE_SINGLE_PASS)), oracle.trace_generate(**tp))
    tp = dict(tp, units_per_group=50, groups=3, topk=20, base=base[:150])
    assert np.array_equal(to_np(trace_on_gpu(kvp, tp)), oracle.trace_generate(**tp))
    assert np.array_equal(to_np(trace_on_gpu(kvp, tp, kvp.TRACE_SINGLE_PASS)), oracle.trace_generate(**tp))


def test_trace_argument_errors(kvp):
    with pytest.raises(kvp.KvpError) as e:
        kvp.trace_generate(1, 16, 4, 17, 0, Q16, 0, 0)          # k > n
    assert e.value.code == kvp.ERR_ARG
    with pytest.raises(kvp.KvpError) as e:
        kvp.trace_generate(1, 16384, 4, 5, 0, Q16, 0, 0)        # group larger than one CTA can hold
    assert e.value.code == kvp.ERR_RANGE
    with pytest.raises(kvp.KvpError) as e:
        kvp.trace_generate(1, 64, 30000, 5, 0, Q16, 1 << 20, 1 << 20)   # random walk could leave int32
    assert e.value.code == kvp.ERR_RANGE
