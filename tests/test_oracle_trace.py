"""Structural and statistical pins of the oracle's synthetic trace generator.

The generator is this repository's own recipe (the paper's traces were recorded from a model),
so beyond these properties its parity is unpinned: the CUDA kernel is compared with it bit by bit.
"""
import numpy as np

from paper_2508_13231_b200 import workloads as wl

Q16 = 65536


def test_exactly_k_bits_per_group_and_step(oracle):
    G, n, S, k = 3, 40, 12, 7           # U = 120: ragged last word
    A = oracle.trace_generate(G, n, S, k, seed=5, rho_q=int(0.9 * Q16), c_q=int(0.43 * Q16), sigma_q=Q16)
    bits = wl.unpack_bits(A, G * n).reshape(S, G, n)
    assert np.all(bits.sum(axis=2) == k)
    assert np.all((A[:, -1] >> np.uint32(120 - 96)) == 0)    # pad bits stay clear


def test_degenerate_noise_selects_by_base_with_ties_to_lower_index(oracle):
    G, n, S, k = 2, 16, 3, 5
    # no noise at all: every score equals base
    A = oracle.trace_generate(G, n, S, k, seed=1, rho_q=Q16, c_q=0, sigma_q=0)
    bits = wl.unpack_bits(A, G * n).reshape(S, G, n)
    assert np.all(bits[:, :, :k] == 1) and np.all(bits[:, :, k:] == 0)      # all equal -> lowest indices
    base = np.array([3, 9, 9, 1, 9, 0, 7, 7, 7, 7, 2, 2, 2, 2, 2, 8] * 2, np.int32) * 1000
    A = oracle.trace_generate(G, n, S, k, seed=1, rho_q=Q16, c_q=0, sigma_q=0, base=base)
    bits = wl.unpack_bits(A, G * n).reshape(S, G, n)
    want = np.zeros(n, np.uint8); want[[1, 2, 4, 15, 6]] = 1               # 9, 9, 9, 8, then the first 7
    assert np.all(bits == want[None, None, :])


def test_noise_is_standardised_and_ar1(oracle):
    G, n, S = 1, 4096, 64
    rho, sigma = 0.9, 1.0
    c = sigma * np.sqrt(1 - rho * rho)
    _, sc = oracle.trace_generate(G, n, S, 16, seed=3, rho_q=int(round(rho * Q16)), c_q=int(round(c * Q16)),
                                  sigma_q=int(round(sigma * Q16)), want_scores=True)
    x = sc.astype(np.float64) / Q16                       # [S][U]
    assert abs(x[0].mean()) < 0.06 and abs(x[0].std() - 1.0) < 0.05       # x_0 ~ N(0, sigma^2), Irwin-Hall(8)
    assert abs(x[-1].std() - 1.0) < 0.05                                   # stationary variance is kept
    lag1 = np.mean([np.corrcoef(x[t], x[t + 1])[0, 1] for t in range(S - 1)])
    assert abs(lag1 - rho) < 0.02
    lag4 = np.mean([np.corrcoef(x[t], x[t + 4])[0, 1] for t in range(S - 4)])
    assert abs(lag4 - rho ** 4) < 0.04
    assert np.abs(x).max() < 6.5                                           # bounded support of Irwin-Hall


def test_higher_rho_means_lower_set_turnover(oracle):
    # "importance variation" (Section IV-B): the accessed set changes less between steps when rho is high
    def turnover(rho):
        c = np.sqrt(1 - rho * rho)
        A = oracle.trace_generate(1, 1024, 32, 100, seed=2, rho_q=int(rho * Q16), c_q=int(c * Q16), sigma_q=Q16)
        b = wl.unpack_bits(A, 1024).astype(np.int32)
        return np.abs(np.diff(b, axis=0)).sum() / 31
    assert turnover(0.99) < turnover(0.9) < turnover(0.5)


def test_bursts_fire_at_the_requested_rate(oracle):
    G, n, S = 1, 8192, 16
    jump = 4 * Q16
    _, s0 = oracle.trace_generate(G, n, S, 8, seed=9, rho_q=Q16, c_q=0, sigma_q=0, want_scores=True)
    _, s1 = oracle.trace_generate(G, n, S, 8, seed=9, rho_q=Q16, c_q=0, sigma_q=0, burst_jump=jump,
                                  burst_thr=int(0.01 * 2 ** 32), want_scores=True)
    assert np.all(s0 == 0)
    fired = np.diff(np.concatenate([np.zeros((1, n), np.int64), s1.astype(np.int64)]), axis=0) // jump
    assert set(np.unique(fired)) <= {0, 1}
    assert abs(fired.mean() - 0.01) < 0.002                  # Bernoulli(0.01) per unit and step; jumps persist (rho = 1)


def test_groups_are_independent(oracle):
    tp = wl.trace_params("layer_8b", seed=0)
    tp = dict(tp, steps=4)
    part = oracle.trace_generate(**tp, group_begin=2, group_count=1)
    small = dict(tp, groups=3, base=tp["base"][: 3 * 2048])
    full = oracle.trace_generate(**small)
    w = 2048 // 32
    assert np.array_equal(part[:, 2 * w:3 * w], full[:, 2 * w:3 * w])
    assert not part[:, :2 * w].any() and not part[:, 3 * w:].any()


def test_named_configurations_have_the_stated_shapes(oracle):
    want = {"tiny": (16, 32, 4, 6), "single_head": (256, 512, 26, 64), "layer_8b": (16384, 256, 256, 4915),
            "full_8b": (524288, 128, 205, 104857), "long_70b": (2621440, 64, 205, 262144)}
    for name, (U, S, k, cap) in want.items():
        cfg = wl.CONFIGS[name]
        assert (wl.units(cfg), cfg["steps"], cfg["topk"], cfg["cap"]) == (U, S, k, cap)
    w = oracle.tick_weights(*wl.CONFIGS["long_70b"]["bw"])
    assert (w["kh"], w["ke"]) == (9, 160)
    w = oracle.tick_weights(*wl.CONFIGS["gh200"]["bw"])
    assert (w["kh"], w["kk"], w["kd"]) == (45, 245, 441)
