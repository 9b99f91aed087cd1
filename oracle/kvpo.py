"""ctypes front end of the CPU oracle (oracle/kvpo.c).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module. It never touches the
CUDA library, and the CUDA library never touches it.

All arrays are numpy arrays on the host; bitmaps are uint32 [steps][ceil(units/32)].
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvpo.c")
_LIB = os.path.join(_HERE, "libkvpo.so")
_lib = None

OK = 0
TABLE_Q = 1024
INIT_STATIC_FIRST, INIT_STATIC_FREQ, INIT_USER = 0, 1, 2
MIG_HBM, MIG_EXT, MIG_PAPER = 1, 2, 3


def build(force=False):
    """Compile kvpo.c into libkvpo.so with gcc (plain -O2, no contraction of a*b+c)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-ffp-contract=off", "-fPIC", "-shared",
             "-o", _LIB, _SRC, "-lm"])
    return _LIB


class AnnealParams(C.Structure):
    _fields_ = [
        ("chains", C.c_uint32), ("levels", C.c_uint32),
        ("moves", C.c_uint64), ("seed", C.c_uint64),
        ("p0", C.c_double), ("alpha", C.c_double),
        ("temps", C.POINTER(C.c_double)),
        ("early_stop_permille", C.c_uint32), ("early_stop_from_level", C.c_uint32),
        ("init_mode", C.c_uint32), ("p_swap_256", C.c_uint32),
        ("max_len_log2", C.c_uint32), ("first_chain", C.c_uint32),
        ("init_schedule", C.POINTER(C.c_uint32)),
    ]


class ChainResult(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in (
        "best_ticks", "best_move", "final_ticks", "moves_done",
        "n_accepted", "n_changed", "n_infeasible", "traj_hash")]

    def astuple(self):
        return tuple(int(getattr(self, n)) for n, _ in self._fields_)


class TraceParams(C.Structure):
    _fields_ = [
        ("groups", C.c_uint32), ("units_per_group", C.c_uint32), ("steps", C.c_uint32), ("topk", C.c_uint32),
        ("seed", C.c_uint64),
        ("rho_q", C.c_int32), ("c_q", C.c_int32), ("sigma_q", C.c_int32), ("burst_jump", C.c_int32),
        ("burst_thr", C.c_uint32), ("reserved", C.c_uint32),
        ("base", C.POINTER(C.c_int32)),
        ("layers", C.c_uint32), ("reserved2", C.c_uint32),
        ("birth", C.POINTER(C.c_uint32)),
    ]


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
        _lib.kvpo_get_weights.restype = C.c_double
    return _lib


def _u32p(a):
    return a.ctypes.data_as(C.POINTER(C.c_uint32)) if a is not None else None


def _u64p(a):
    return a.ctypes.data_as(C.POINTER(C.c_uint64)) if a is not None else None


def _chk(rc, what):
    if rc != OK:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def philox(ctr, key):
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    lib().kvpo_philox4x32_10(c, k, o)
    return tuple(int(x) for x in o)


def tick_weights(bw_hbm, bw_link, bw_dram):
    """-> dict(kh, kk, kd, ke, lcm, gcd)"""
    o = (C.c_uint64 * 6)()
    _chk(lib().kvpo_tick_weights(C.c_uint64(bw_hbm), C.c_uint64(bw_link), C.c_uint64(bw_dram), o), "tick_weights")
    return dict(zip(("kh", "kk", "kd", "ke", "lcm", "gcd"), (int(x) for x in o)))


class Problem:
    def __init__(self, units, bytes_per_unit, steps, access, cap, bw_hbm, bw_link, bw_dram,
                 mig_flags=MIG_PAPER, hw=None, ew=None, birth=None):
        access = np.ascontiguousarray(access, dtype=np.uint32)
        self.units, self.steps, self.cap = int(units), int(steps), int(cap)
        self.w32 = (self.units + 31) // 32
        assert access.size == self.steps * self.w32
        self.access = access.reshape(self.steps, self.w32)
        hw = None if hw is None else np.ascontiguousarray(hw, dtype=np.uint32)
        ew = None if ew is None else np.ascontiguousarray(ew, dtype=np.uint32)
        self._h = C.c_void_p()
        rc = lib().kvpo_create(C.byref(self._h), C.c_uint32(units), C.c_uint64(bytes_per_unit), C.c_uint32(steps),
                               _u32p(self.access), C.c_uint32(cap), C.c_uint64(bw_hbm), C.c_uint64(bw_link),
                               C.c_uint64(bw_dram), C.c_uint32(mig_flags), _u32p(hw), _u32p(ew))
        _chk(rc, "create")
        o = (C.c_uint64 * 6)()
        self.seconds_per_tick = float(lib().kvpo_get_weights(self._h, o))
        self.weights = dict(zip(("kh", "kk", "kd", "ke", "lcm", "gcd"), (int(x) for x in o)))
        self.birth = None
        if birth is not None:
            self.birth = np.ascontiguousarray(birth, dtype=np.uint32)
            assert self.birth.size == self.units
            _chk(lib().kvpo_set_births(self._h, _u32p(self.birth)), "set_births")

    def __del__(self):
        if getattr(self, "_h", None) is not None and self._h and lib is not None:   # lib is None at interpreter exit
            lib().kvpo_destroy(self._h)
            self._h = None

    def _sched(self, P):
        P = np.ascontiguousarray(P, dtype=np.uint32)
        assert P.size == self.steps * self.w32
        return P

    def eval(self, P):
        """-> dict(step_ticks, total_ticks, step_seconds, total_seconds, bad_step, counts[S][4])"""
        P = self._sched(P)
        st = np.zeros(self.steps, np.uint64)
        ss = np.zeros(self.steps, np.float64)
        cnt = np.zeros((self.steps, 4), np.uint32)
        tt = C.c_uint64(); ts = C.c_double(); bad = C.c_int32()
        _chk(lib().kvpo_eval(self._h, _u32p(P), _u64p(st), C.byref(tt), ss.ctypes.data_as(C.POINTER(C.c_double)),
                             C.byref(ts), C.byref(bad), _u32p(cnt)), "eval")
        hb = np.zeros(self.steps, np.uint32)
        _chk(lib().kvpo_eval_hb(self._h, _u32p(P), _u32p(hb)), "eval_hb")
        return dict(step_ticks=st, total_ticks=int(tt.value), step_seconds=ss, total_seconds=float(ts.value),
                    bad_step=int(bad.value), counts=cnt, hb=hb)

    def init_placement(self, mode):
        P = np.zeros((self.steps, self.w32), np.uint32)
        _chk(lib().kvpo_init_placement(self._h, C.c_uint32(mode), _u32p(P)), "init_placement")
        return P

    def make_params(self, chains, moves, seed=0, levels=64, p0=0.8, alpha=0.9, temps=None,
                    early_stop_permille=0, early_stop_from_level=0, init_mode=INIT_STATIC_FREQ,
                    p_swap_256=128, max_len_log2=5, init_schedule=None, first_chain=0):
        ap = AnnealParams()
        ap.chains, ap.levels, ap.moves, ap.seed = chains, levels, moves, seed
        ap.p0, ap.alpha = p0, alpha
        keep = []
        if temps is not None:
            t = np.ascontiguousarray(temps, dtype=np.float64)
            assert t.size == levels
            keep.append(t)
            ap.temps = t.ctypes.data_as(C.POINTER(C.c_double))
        ap.early_stop_permille, ap.early_stop_from_level = early_stop_permille, early_stop_from_level
        ap.init_mode, ap.p_swap_256, ap.max_len_log2 = init_mode, p_swap_256, max_len_log2
        ap.first_chain = first_chain
        if init_schedule is not None:
            s = self._sched(init_schedule)
            keep.append(s)
            ap.init_schedule = _u32p(s)
        ap._keep = keep
        return ap

    def temps(self, ap):
        """Temperature ladder the parameters imply -> (temps[levels], calibration mean delta)."""
        if ap.temps:
            return np.ctypeslib.as_array(ap.temps, shape=(ap.levels,)).copy(), 0
        t = np.zeros(ap.levels, np.float64)
        mean = C.c_uint64()
        _chk(lib().kvpo_default_temps(self._h, C.byref(ap), t.ctypes.data_as(C.POINTER(C.c_double)), C.byref(mean)),
             "default_temps")
        return t, int(mean.value)

    def anneal_chains(self, ap, chain_begin, chain_count, upto_moves=None, want_final=False, want_best=False,
                      table=None, shifts=None):
        """-> (list of ChainResult, final_states or None, best_states or None)"""
        if table is None:
            t, _ = self.temps(ap)
            table, shifts = accept_table(t)
        res = (ChainResult * chain_count)()
        fin = np.zeros((chain_count, self.steps, self.w32), np.uint32) if want_final else None
        bst = np.zeros((chain_count, self.steps, self.w32), np.uint32) if want_best else None
        upto = ap.moves if upto_moves is None else upto_moves
        _chk(lib().kvpo_anneal_chains(self._h, C.byref(ap), _u32p(table), _u32p(shifts), C.c_uint32(chain_begin),
                                      C.c_uint32(chain_count), C.c_uint64(upto), res, _u32p(fin), _u32p(bst)),
             "anneal_chains")
        return list(res), fin, bst

    def anneal(self, ap, table=None, shifts=None):
        """-> dict(best_schedule, best_ticks, best_seconds, best_chain, per_chain)"""
        if table is None:
            t, _ = self.temps(ap)
            table, shifts = accept_table(t)
        res = (ChainResult * ap.chains)()
        best = np.zeros((self.steps, self.w32), np.uint32)
        bt = C.c_uint64(); bc = C.c_uint32()
        _chk(lib().kvpo_anneal(self._h, C.byref(ap), _u32p(table), _u32p(shifts), _u32p(best), C.byref(bt),
                               C.byref(bc), res), "anneal")
        return dict(best_schedule=best, best_ticks=int(bt.value), best_seconds=int(bt.value) * self.seconds_per_tick,
                    best_chain=int(bc.value), per_chain=list(res))

    def decode_moves(self, ap, chain, m_begin, count, tag=1):
        """The proposals of moves m_begin .. m_begin+count-1 of `chain` -> uint32 [count][6] = (swap, s0, len, u, v, w).
        tag 1 = the annealer's moves, 2 = the calibration proposals."""
        out = np.zeros((count, 6), np.uint32)
        _chk(lib().kvpo_decode_moves(self._h, C.byref(ap), C.c_uint32(chain), C.c_uint32(tag), C.c_uint64(m_begin),
                                     C.c_uint32(count), _u32p(out)), "decode_moves")
        return out

    def exchange_tables(self, ap, rungs):
        """Ladder temperatures, move table and exchange table of a replica-exchange run (ap.levels == rungs).
        -> dict(temps, table, shifts, pair_temps, xalways, xtable, xshifts)"""
        assert ap.levels == rungs
        temps, _ = self.temps(ap)
        table, shifts = accept_table(temps)
        pair = np.ones(max(1, rungs - 1), np.float64)
        always = np.zeros(max(1, rungs - 1), np.uint32)
        _chk(lib().kvpo_exchange_temps(temps.ctypes.data_as(C.POINTER(C.c_double)), C.c_uint32(rungs),
                                       pair.ctypes.data_as(C.POINTER(C.c_double)), _u32p(always)), "exchange_temps")
        xtable, xshifts = accept_table(pair)
        return dict(temps=temps, table=table, shifts=shifts, pair_temps=pair, xalways=always, xtable=xtable, xshifts=xshifts)

    def anneal_exchange(self, ap, rungs, every, want_log=False, want_samples=False, want_best=False):
        """Replica exchange: ap.chains chains in ladders of `rungs`, exchanges every `every` moves.
        -> dict(per_chain, final_rung, n_exchanged, best_ticks, best_chain, xlog [rounds][ladders][rungs-1][3] or None,
                samples [rounds][chains][2] or None)"""
        tb = self.exchange_tables(ap, rungs)
        n = ap.chains
        res = (ChainResult * n)()
        final_rung = np.zeros(n, np.uint32)
        n_ex = np.zeros(n, np.uint32)
        rounds = (ap.moves + every - 1) // every
        ladders = n // rungs
        xlog = np.zeros((rounds, ladders, max(1, rungs - 1), 3), np.uint64) if want_log else None
        samples = np.zeros((rounds, n, 2), np.uint64) if want_samples else None
        bst = np.zeros((n, self.steps, self.w32), np.uint32) if want_best else None
        _chk(lib().kvpo_anneal_exchange(self._h, C.byref(ap), C.c_uint32(rungs), C.c_uint64(every), _u32p(tb["table"]),
                                        _u32p(tb["shifts"]), _u32p(tb["xalways"]), _u32p(tb["xtable"]), _u32p(tb["xshifts"]),
                                        res, _u32p(final_rung), _u32p(n_ex), _u64p(xlog), _u64p(samples), _u32p(bst)), "anneal_exchange")
        per = list(res)
        ticks = [r.best_ticks for r in per]
        bc = int(np.argmin(ticks))
        return dict(per_chain=per, final_rung=final_rung, n_exchanged=n_ex, best_ticks=int(ticks[bc]),
                    best_chain=ap.first_chain + bc, xlog=xlog, samples=samples, tables=tb,
                    best_schedule=bst[bc] if want_best else None)

    def check_total(self, P, ticks):
        return lib().kvpo_check_total(self._h, _u32p(self._sched(P)), C.c_uint64(ticks)) == 0


def accept_table(temps):
    temps = np.ascontiguousarray(temps, dtype=np.float64)
    levels = temps.size
    table = np.zeros((levels, TABLE_Q), np.uint32)
    shifts = np.zeros(levels, np.uint32)
    _chk(lib().kvpo_accept_table(temps.ctypes.data_as(C.POINTER(C.c_double)), C.c_uint32(levels),
                                 _u32p(table), _u32p(shifts)), "accept_table")
    return table, shifts


def trace_generate(groups, units_per_group, steps, topk, seed, rho_q, c_q, sigma_q, burst_jump=0, burst_thr=0,
                   base=None, group_begin=0, group_count=None, want_scores=False, layers=0, birth=None):
    """-> access [steps][W32] (and scores [steps][U] int32 when want_scores)."""
    tp = TraceParams()
    tp.layers = layers
    if birth is not None:
        birth = np.ascontiguousarray(birth, dtype=np.uint32)
        assert birth.size == groups * units_per_group
        tp.birth = birth.ctypes.data_as(C.POINTER(C.c_uint32))
    tp.groups, tp.units_per_group, tp.steps, tp.topk, tp.seed = groups, units_per_group, steps, topk, seed
    tp.rho_q, tp.c_q, tp.sigma_q, tp.burst_jump, tp.burst_thr = rho_q, c_q, sigma_q, burst_jump, burst_thr
    if base is not None:
        base = np.ascontiguousarray(base, dtype=np.int32)
        assert base.size == groups * units_per_group
        tp.base = base.ctypes.data_as(C.POINTER(C.c_int32))
    U = groups * units_per_group
    w32 = (U + 31) // 32
    acc = np.zeros((steps, w32), np.uint32)
    sc = np.zeros((steps, U), np.int32) if want_scores else None
    if group_count is None:
        group_count = groups - group_begin
    _chk(lib().kvpo_trace_generate(C.byref(tp), C.c_uint32(group_begin), C.c_uint32(group_count), _u32p(acc),
                                   sc.ctypes.data_as(C.POINTER(C.c_int32)) if want_scores else None),
         "trace_generate")
    return (acc, sc) if want_scores else acc


class WRParams(C.Structure):
    _fields_ = [("chains", C.c_uint32), ("levels", C.c_uint32), ("iters", C.c_uint64), ("seed", C.c_uint64),
                ("p0", C.c_double), ("alpha", C.c_double), ("early_stop_permille", C.c_uint32),
                ("w0", C.c_uint32), ("r0", C.c_uint32), ("reserved", C.c_uint32)]


class WRResult(C.Structure):
    _fields_ = [("best_ticks", C.c_uint64), ("final_ticks", C.c_uint64), ("iters_done", C.c_uint64),
                ("n_accepted", C.c_uint64), ("best_w", C.c_uint32), ("best_r", C.c_uint32),
                ("final_w", C.c_uint32), ("final_r", C.c_uint32)]

    def astuple(self):
        return tuple(int(getattr(self, n)) for n, _ in self._fields_)


def policy_lookahead(prob, window, ratio_permille, init_mode=INIT_STATIC_FIRST):
    """Schedule of the look-ahead policy (W = window steps, R = ratio_permille / 1000) -> uint32 [S][W32]."""
    P = np.zeros((prob.steps, prob.w32), np.uint32)
    _chk(lib().kvpo_policy_lookahead(prob._h, C.c_uint32(init_mode), C.c_uint32(window), C.c_uint32(ratio_permille),
                                     _u32p(P)), "policy_lookahead")
    return P


def policy_reactive(prob, init_mode=INIT_STATIC_FIRST):
    """Schedule of promote-on-miss with LRU eviction -> uint32 [S][W32]."""
    P = np.zeros((prob.steps, prob.w32), np.uint32)
    _chk(lib().kvpo_policy_reactive(prob._h, C.c_uint32(init_mode), _u32p(P)), "policy_reactive")
    return P


def wr_grid(prob, w_max, n_ratio=11, init_mode=INIT_STATIC_FIRST):
    """T(W, R) in ticks for W = 1..w_max, R = r / (n_ratio - 1) -> uint64 [w_max][n_ratio]."""
    T = np.zeros((w_max, n_ratio), np.uint64)
    for w in range(1, w_max + 1):
        for r in range(n_ratio):
            T[w - 1, r] = prob.eval(policy_lookahead(prob, w, (1000 * r) // (n_ratio - 1), init_mode))["total_ticks"]
    return T


def wr_params(chains, iters, seed=0, levels=16, p0=0.8, alpha=0.9, early_stop_permille=0, w0=1, r0=0):
    wp = WRParams()
    wp.chains, wp.levels, wp.iters, wp.seed = chains, levels, iters, seed
    wp.p0, wp.alpha, wp.early_stop_permille, wp.w0, wp.r0 = p0, alpha, early_stop_permille, w0, r0
    return wp


def wr_temps(table, wp):
    table = np.ascontiguousarray(table, dtype=np.uint64)
    t = np.zeros(wp.levels, np.float64)
    mean = C.c_uint64()
    _chk(lib().kvpo_wr_temps(_u64p(table), C.c_uint32(table.shape[0]), C.c_uint32(table.shape[1]), C.byref(wp),
                             t.ctypes.data_as(C.POINTER(C.c_double)), C.byref(mean)), "wr_temps")
    return t, int(mean.value)


def wr_anneal(table, wp):
    """The paper's (W, R) annealer on a latency table -> list of WRResult, one per chain."""
    table = np.ascontiguousarray(table, dtype=np.uint64)
    temps, _ = wr_temps(table, wp)
    acc, shifts = accept_table(temps)
    res = (WRResult * wp.chains)()
    _chk(lib().kvpo_wr_anneal(_u64p(table), C.c_uint32(table.shape[0]), C.c_uint32(table.shape[1]), C.byref(wp),
                              _u32p(acc), _u32p(shifts), res), "wr_anneal")
    return list(res)


def policy_page(prob, page_units):
    """Schedule of page-granularity placement with perfect foresight of the current step -> uint32 [S][W32]."""
    P = np.zeros((prob.steps, prob.w32), np.uint32)
    _chk(lib().kvpo_policy_page(prob._h, C.c_uint32(page_units), _u32p(P)), "policy_page")
    return P
