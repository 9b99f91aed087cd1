"""kvp_eval_noalloc against kvp_eval.

Some users of the library cannot allocate device memory when they score schedules: a loop that must not
stall on cudaMalloc, or a process in which a framework's pool already owns the GPU's memory. For them
the library offers an entry point whose scratch is a fixed 1 MiB array inside the library. This test calls
it through the C ABI twice in a row (the second call finds the first call's leftovers in the shared
scratch) and expects exactly kvp_eval's numbers: ticks and flags bit for bit, seconds within 1e-9 relative.
The file sorts last so that a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2508_13231_b200 import workloads as wl
from gpu_util import to_dev

pytestmark = pytest.mark.gpu
GB = 10 ** 9


def _outputs(n, S):
    return dict(step_ticks=torch.full((n, S), -1, dtype=torch.int64, device="cuda"),
                total_ticks=torch.full((n,), -1, dtype=torch.int64, device="cuda"),
                step_seconds=torch.full((n, S), -1.0, dtype=torch.float64, device="cuda"),
                total_seconds=torch.full((n,), -1.0, dtype=torch.float64, device="cuda"),
                bad_step=torch.full((n,), -7, dtype=torch.int32, device="cuda"))


# one shape per counting kernel: rows of 8 words (sub-warp groups) and rows of 512 words (warp per chunk,
# accumulated with atomics into scratch that the call must clear itself)
@pytest.mark.parametrize("U,S,n1,n2", [(256, 512, 5, 3), (16384, 64, 6, 9), (1000, 33, 40, 2)])
def test_noalloc_matches_eval_twice_in_a_row(oracle, U, S, n1, n2):
    from paper_2508_13231_b200 import kvp
    cap = U // 4
    A = wl.random_access(U, S, 0.2, seed=U)
    hw, ew = np.arange(S) % 2, np.arange(S) % 3
    prob = kvp.Problem(U, 8192, S, to_dev(A), cap, 8000 * GB, 900 * GB, 900 * GB, hw=hw, ew=ew)
    ref = oracle.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB, hw=hw, ew=ew)
    for call, n in enumerate((n1, n2)):
        scheds = wl.random_schedules(U, S, cap, n, seed=100 + call, churn=0.1)
        bits = wl.unpack_bits(scheds[-1], U); bits[S // 2, :cap + 1] = 1       # one schedule over capacity
        scheds[-1] = wl.pack_bits(bits)
        dev = to_dev(scheds)
        want = prob.eval(dev)
        got = _outputs(n, S)
        prob.eval_noalloc(dev, **got)
        torch.cuda.synchronize()
        assert torch.equal(got["step_ticks"], want["step_ticks"]), call
        assert torch.equal(got["total_ticks"], want["total_ticks"]), call
        assert torch.equal(got["bad_step"], want["bad_step"]), call
        assert int(got["bad_step"][-1]) == S // 2
        assert torch.allclose(got["step_seconds"], want["step_seconds"], rtol=1e-9, atol=0)
        assert torch.allclose(got["total_seconds"], want["total_seconds"], rtol=1e-9, atol=0)
        # and directly against the oracle, so that this file stands on its own: first and last schedule of the batch
        for i in (0, n - 1):
            o = ref.eval(scheds[i])
            assert np.array_equal(got["step_ticks"][i].cpu().numpy().view(np.uint64), o["step_ticks"]), (call, i)
            assert int(got["total_ticks"][i]) == o["total_ticks"] and int(got["bad_step"][i]) == o["bad_step"]
            assert float(got["total_seconds"][i]) == pytest.approx(o["total_seconds"], rel=1e-9)


def test_noalloc_refuses_batches_beyond_its_scratch():
    from paper_2508_13231_b200 import kvp
    U, S = 64, 1024
    A = wl.random_access(U, S, 0.2, seed=1)
    prob = kvp.Problem(U, 8192, S, to_dev(A), 16, 8000 * GB, 900 * GB, 900 * GB)
    n_ok = kvp.NOALLOC_SCRATCH_BYTES // (16 * S)          # 64 schedules of 1024 steps fill the 1 MiB exactly
    scheds = to_dev(np.zeros((n_ok + 1, S, 2), np.uint32))
    out = _outputs(n_ok + 1, S)
    with pytest.raises(kvp.KvpError) as e:
        prob.eval_noalloc(scheds, **out)
    assert e.value.code == kvp.ERR_RANGE
    torch.cuda.synchronize()
    assert int(out["total_ticks"][0]) == -1               # nothing was launched
    ok = {k: v[:n_ok] for k, v in out.items()}
    prob.eval_noalloc(scheds[:n_ok], **ok)
    torch.cuda.synchronize()
    assert torch.equal(ok["total_ticks"], prob.eval(scheds[:n_ok])["total_ticks"])


def test_noalloc_serves_the_largest_batch_its_scratch_admits(oracle):
    """One-step schedules: the limit admits 65,536 of them, more than one launch can index, so the call goes in
    slices. Compared with kvp_eval on all of them and with the oracle on a few, twice in a row."""
    from paper_2508_13231_b200 import kvp
    U, S, cap = 96, 1, 40
    A = wl.random_access(U, S, 0.3, seed=5)
    prob = kvp.Problem(U, 8192, S, to_dev(A), cap, 8000 * GB, 900 * GB, 900 * GB)
    ref = oracle.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB)
    n = kvp.NOALLOC_SCRATCH_BYTES // 16
    assert n == 65536
    rng = np.random.Generator(np.random.PCG64(11))
    scheds = (rng.integers(0, 2 ** 32, (n, S, 3), dtype=np.uint64) & rng.integers(0, 2 ** 32, (n, S, 3), dtype=np.uint64)
              & rng.integers(0, 2 ** 32, (n, S, 3), dtype=np.uint64)).astype(np.uint32)
    dev = to_dev(scheds)
    want = prob.eval(dev)
    for call in range(2):
        got = _outputs(n, S)
        prob.eval_noalloc(dev, **got)
        torch.cuda.synchronize()
        assert torch.equal(got["step_ticks"], want["step_ticks"]) and torch.equal(got["total_ticks"], want["total_ticks"])
        assert torch.equal(got["bad_step"], want["bad_step"])
        for i in (0, 32767, 32768, 50000, n - 1):
            o = ref.eval(scheds[i])
            assert int(got["total_ticks"][i]) == o["total_ticks"] and int(got["bad_step"][i]) == o["bad_step"], i
