"""Thin ctypes binding of libkvp.so (include/kvp.h): argument marshalling only.

Bulk data are torch CUDA tensors (device memory and streams come from PyTorch); every step of the
computation runs in the library's CUDA kernels. There is no CPU path: if the shared library is
missing or no CUDA device is usable, calls raise.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkvp.so")

OK = 0
ERR_ARG, ERR_CAPACITY, ERR_RANGE, ERR_CUDA, ERR_NOMEM, ERR_TIMEOUT, ERR_INTERNAL = -1, -2, -3, -4, -5, -6, -7
MIG_HBM, MIG_EXT, MIG_PAPER = 1, 2, 3
INIT_STATIC_FIRST, INIT_STATIC_FREQ, INIT_USER = 0, 1, 2
TABLE_Q = 1024

NOALLOC_SCRATCH_BYTES = 1 << 20

EXPORTS = [
    "kvp_create", "kvp_destroy", "kvp_get_info", "kvp_eval", "kvp_eval_counts", "kvp_eval_noalloc", "kvp_accept_table", "kvp_anneal",
    "kvp_anneal_chain_state", "kvp_trace_generate", "kvp_philox4x32_10", "kvp_strerror", "kvp_last_cuda_error",
    "kvp_policy_lookahead", "kvp_policy_reactive", "kvp_policy_page", "kvp_wr_grid", "kvp_wr_anneal", "kvp_set_births",
    "kvp_set_test_hooks", "kvp_anneal_exchange", "kvp_exchange_temps",
]


class KvpError(RuntimeError):
    def __init__(self, code, what):
        self.code = code
        msg = f"{what}: {_lib().kvp_strerror(code).decode()} ({code})"
        if code in (ERR_CUDA, ERR_NOMEM):
            msg += " [" + _lib().kvp_last_cuda_error().decode() + "]"
        super().__init__(msg)


class MemSys(C.Structure):
    _fields_ = [("bw_hbm", C.c_uint64), ("bw_link", C.c_uint64), ("bw_dram", C.c_uint64),
                ("mig_flags", C.c_uint32), ("reserved", C.c_uint32)]


class Info(C.Structure):
    _fields_ = [("kappa_h", C.c_uint64), ("kappa_k", C.c_uint64), ("kappa_d", C.c_uint64), ("kappa_e", C.c_uint64),
                ("lcm", C.c_uint64), ("gcd", C.c_uint64), ("seconds_per_tick", C.c_double),
                ("units", C.c_uint32), ("steps", C.c_uint32), ("words_per_row", C.c_uint32), ("capacity", C.c_uint32)]


class AnnealParams(C.Structure):
    _fields_ = [
        ("chains", C.c_uint32), ("levels", C.c_uint32), ("moves", C.c_uint64), ("seed", C.c_uint64),
        ("p0", C.c_double), ("alpha", C.c_double), ("temps", C.POINTER(C.c_double)),
        ("early_stop_permille", C.c_uint32), ("early_stop_from_level", C.c_uint32),
        ("init_mode", C.c_uint32), ("p_swap_256", C.c_uint32), ("max_len_log2", C.c_uint32), ("first_chain", C.c_uint32),
        ("init_schedule", C.c_void_p),
    ]


class ChainResult(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in (
        "best_ticks", "best_move", "final_ticks", "moves_done", "n_accepted", "n_changed", "n_infeasible", "traj_hash")]

    def astuple(self):
        return tuple(int(getattr(self, n)) for n, _ in self._fields_)


class AnnealStats(C.Structure):
    _fields_ = [
        ("init_ticks", C.c_uint64), ("best_ticks", C.c_uint64), ("best_chain", C.c_uint32), ("levels", C.c_uint32),
        ("best_move", C.c_uint64), ("moves_total", C.c_uint64), ("calib_mean_delta", C.c_uint64), ("temp0", C.c_double),
        ("winner_hits", C.c_uint64), ("winner_accessed", C.c_uint64),
        ("ms_init", C.c_float), ("ms_chains", C.c_float), ("ms_finish", C.c_float), ("kernel_launches", C.c_uint32),
        ("per_chain", C.POINTER(ChainResult)), ("chain_launches", C.c_uint32), ("resident_chains", C.c_uint32),
        ("wide_kernel", C.c_uint32), ("reserved", C.c_uint32),
        ("work_again", C.c_uint64), ("work_listed", C.c_uint64), ("work_items", C.c_uint64),
        ("exchanges_tried", C.c_uint64), ("exchanges_accepted", C.c_uint64), ("exchange_rounds", C.c_uint32),
        ("reserved2", C.c_uint32),
    ]


class ExchangeParams(C.Structure):
    _fields_ = [("rungs", C.c_uint32), ("reserved", C.c_uint32), ("exchange_every", C.c_uint64)]


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


class TraceParams(C.Structure):
    _fields_ = [
        ("groups", C.c_uint32), ("units_per_group", C.c_uint32), ("steps", C.c_uint32), ("topk", C.c_uint32),
        ("seed", C.c_uint64), ("rho_q", C.c_int32), ("c_q", C.c_int32), ("sigma_q", C.c_int32), ("burst_jump", C.c_int32),
        ("burst_thr", C.c_uint32), ("flags", C.c_uint32), ("base", C.c_void_p),
        ("layers", C.c_uint32), ("reserved", C.c_uint32), ("birth", C.c_void_p),
    ]


class TestHooks(C.Structure):
    _fields_ = [("warps_per_chain", C.c_uint32), ("drop_turn", C.c_uint32), ("split_queue_plus1", C.c_uint32),
                ("resident", C.c_uint32), ("overlay", C.c_uint32)]


_handle = None


def _lib():
    global _handle
    if _handle is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2508_13231_b200.build` "
                              "(there is no CPU fallback)")
        h = C.CDLL(LIB_PATH)
        h.kvp_strerror.restype = C.c_char_p
        h.kvp_last_cuda_error.restype = C.c_char_p
        h.kvp_destroy.restype = None
        h.kvp_philox4x32_10.restype = None
        h.kvp_set_test_hooks.restype = None
        _handle = h
    return _handle


def _chk(rc, what):
    if rc != OK:
        raise KvpError(rc, what)


def _ptr(t, dtype=None):
    if t is None:
        return C.c_void_p(0)
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def set_test_hooks(warps_per_chain=0, drop_turn=0, split_queue=None, resident=0, overlay=0):
    """kvp_set_test_hooks (test-suite and tuning only; process-wide). Called without arguments it resets everything."""
    h = TestHooks(int(warps_per_chain), int(drop_turn), 0 if split_queue is None else int(split_queue) + 1, int(resident),
                  int(overlay))
    _lib().kvp_set_test_hooks(C.byref(h))


def philox(ctr, key):
    c = (C.c_uint32 * 4)(*ctr); k = (C.c_uint32 * 2)(*key); o = (C.c_uint32 * 4)()
    _lib().kvp_philox4x32_10(c, k, o)
    return tuple(int(x) for x in o)


def accept_table(temps):
    """Host-side acceptance thresholds -> (table [levels][1024], shifts [levels]) as CPU int32 tensors holding the uint32 words."""
    temps = torch.as_tensor(temps, dtype=torch.float64).contiguous().cpu()
    levels = temps.numel()
    table = torch.zeros((levels, TABLE_Q), dtype=torch.int32)
    shifts = torch.zeros(levels, dtype=torch.int32)
    _chk(_lib().kvp_accept_table(C.c_void_p(temps.data_ptr()), C.c_uint32(levels), C.c_void_p(table.data_ptr()),
                                 C.c_void_p(shifts.data_ptr())), "kvp_accept_table")
    return table, shifts


TRACE_SINGLE_PASS = 1


def trace_generate(groups, units_per_group, steps, topk, seed, rho_q, c_q, sigma_q, burst_jump=0, burst_thr=0,
                   base=None, out=None, stream=None, flags=0, layers=0, birth=None):
    """Synthetic access bitmaps on the current CUDA device -> int32 tensor [steps][ceil(U/32)] (bit pattern uint32).

    layers: the steps are (token, layer) pairs; birth: int32 CUDA tensor [U] of the steps at which units appear."""
    tp = TraceParams()
    tp.layers = layers
    if birth is not None:
        if birth.numel() != groups * units_per_group:
            raise ValueError("birth must have one entry per unit")
        tp.birth = _ptr(birth, torch.int32)
    tp.groups, tp.units_per_group, tp.steps, tp.topk, tp.seed = groups, units_per_group, steps, topk, seed
    tp.rho_q, tp.c_q, tp.sigma_q, tp.burst_jump, tp.burst_thr = rho_q, c_q, sigma_q, burst_jump, burst_thr
    tp.flags = flags
    if base is not None:
        if base.numel() != groups * units_per_group:
            raise ValueError("base must have one entry per unit")
        tp.base = _ptr(base, torch.int32)
    w32 = (groups * units_per_group + 31) // 32
    if out is None:
        out = torch.empty((steps, w32), dtype=torch.int32, device="cuda")
    _chk(_lib().kvp_trace_generate(C.byref(tp), _ptr(out, torch.int32), _stream(stream)), "kvp_trace_generate")
    return out


class Problem:
    """A problem instance (kvp_create). Bitmaps are int32 CUDA tensors holding the uint32 words."""

    def __init__(self, units, bytes_per_unit, steps, access, cap, bw_hbm, bw_link, bw_dram, mig_flags=MIG_PAPER,
                 hw=None, ew=None, stream=None, birth=None):
        self.units, self.steps, self.cap = int(units), int(steps), int(cap)
        self.w32 = (self.units + 31) // 32
        if access.numel() != self.steps * self.w32:
            raise ValueError("access bitmap has the wrong size")
        ms = MemSys(int(bw_hbm), int(bw_link), int(bw_dram), int(mig_flags), 0)
        hw_a = (C.c_uint32 * steps)(*[int(x) for x in hw]) if hw is not None else None
        ew_a = (C.c_uint32 * steps)(*[int(x) for x in ew]) if ew is not None else None
        self._h = C.c_void_p()
        _chk(_lib().kvp_create(C.byref(self._h), C.c_uint32(units), C.c_uint64(bytes_per_unit), C.c_uint32(steps),
                               _ptr(access, torch.int32), C.c_uint32(cap), C.byref(ms), hw_a, ew_a, _stream(stream)),
             "kvp_create")
        if birth is not None:                                # growing cache (kvp_set_births)
            if birth.numel() != self.units:
                self.close()
                raise ValueError("birth must have one entry per unit")
            rc = _lib().kvp_set_births(self._h, _ptr(birth, torch.int32), _stream(stream))
            if rc:
                self.close()
                _chk(rc, "kvp_set_births")
        info = Info()
        _chk(_lib().kvp_get_info(self._h, C.byref(info)), "kvp_get_info")
        self.info = info
        self.seconds_per_tick = float(info.seconds_per_tick)
        self.weights = dict(kh=int(info.kappa_h), kk=int(info.kappa_k), kd=int(info.kappa_d), ke=int(info.kappa_e),
                            lcm=int(info.lcm), gcd=int(info.gcd))

    def close(self):
        if getattr(self, "_h", None):
            _lib().kvp_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _n(self, schedules):
        per = self.steps * self.w32
        if schedules.numel() % per:
            raise ValueError("schedules must be [n][steps][W32]")
        return schedules.numel() // per

    def eval(self, schedules, want_steps=True, want_seconds=True, stream=None):
        """kvp_eval -> dict of CUDA tensors (step_ticks int64 [n][S], total_ticks int64 [n], seconds, bad_step)."""
        n = self._n(schedules)
        dev = schedules.device
        st = torch.empty((n, self.steps), dtype=torch.int64, device=dev) if want_steps else None
        tt = torch.empty(n, dtype=torch.int64, device=dev)
        ss = torch.empty((n, self.steps), dtype=torch.float64, device=dev) if (want_steps and want_seconds) else None
        ts = torch.empty(n, dtype=torch.float64, device=dev) if want_seconds else None
        bad = torch.empty(n, dtype=torch.int32, device=dev)
        _chk(_lib().kvp_eval(self._h, _ptr(schedules, torch.int32), C.c_uint32(n), _ptr(st), _ptr(tt), _ptr(ss),
                             _ptr(ts), _ptr(bad), _stream(stream)), "kvp_eval")
        return dict(step_ticks=st, total_ticks=tt, step_seconds=ss, total_seconds=ts, bad_step=bad)

    def eval_noalloc(self, schedules, step_ticks, total_ticks, step_seconds, total_seconds, bad_step, stream=None):
        """kvp_eval_noalloc: like eval(), but the library allocates nothing. The caller passes every output
        tensor (CUDA; any but total_ticks may be None) so that this wrapper allocates nothing either.
        For code that cannot call the allocator here: a latency-bound loop, or a process whose memory pool
        owns the device. Batches are limited to n * steps <= 65536; calls share one scratch array per GPU,
        so do not let two of them run concurrently."""
        n = self._n(schedules)
        _chk(_lib().kvp_eval_noalloc(self._h, _ptr(schedules, torch.int32), C.c_uint32(n), _ptr(step_ticks),
                                     _ptr(total_ticks), _ptr(step_seconds), _ptr(total_seconds), _ptr(bad_step),
                                     _stream(stream)), "kvp_eval_noalloc")

    def eval_counts(self, schedules, stream=None):
        n = self._n(schedules)
        cnt = torch.empty((n, self.steps, 4), dtype=torch.int32, device=schedules.device)
        _chk(_lib().kvp_eval_counts(self._h, _ptr(schedules, torch.int32), C.c_uint32(n), _ptr(cnt), _stream(stream)),
             "kvp_eval_counts")
        return cnt

    def make_params(self, chains, moves, seed=0, levels=64, p0=0.8, alpha=0.9, temps=None, early_stop_permille=0,
                    early_stop_from_level=0, init_mode=INIT_STATIC_FREQ, p_swap_256=128, max_len_log2=5,
                    init_schedule=None, first_chain=0):
        ap = AnnealParams()
        ap.chains, ap.levels, ap.moves, ap.seed = chains, levels, moves, seed
        ap.p0, ap.alpha = p0, alpha
        keep = []
        if temps is not None:
            arr = (C.c_double * levels)(*[float(x) for x in temps])
            keep.append(arr)
            ap.temps = C.cast(arr, C.POINTER(C.c_double))
        ap.early_stop_permille, ap.early_stop_from_level = early_stop_permille, early_stop_from_level
        ap.init_mode, ap.p_swap_256, ap.max_len_log2 = init_mode, p_swap_256, max_len_log2
        ap.first_chain = first_chain
        if init_schedule is not None:
            keep.append(init_schedule)
            ap.init_schedule = _ptr(init_schedule, torch.int32)
        ap._keep = keep
        return ap

    def anneal(self, ap, want_schedule=True, want_per_chain=False, stream=None):
        """kvp_anneal -> dict(best_schedule (CUDA int32 [S][W32]), best_ticks, best_seconds, stats, per_chain)."""
        best = torch.empty((self.steps, self.w32), dtype=torch.int32, device="cuda") if want_schedule else None
        bt = C.c_uint64(); bs = C.c_double()
        stats = AnnealStats()
        per = (ChainResult * ap.chains)() if want_per_chain else None
        if per is not None:
            stats.per_chain = C.cast(per, C.POINTER(ChainResult))
        _chk(_lib().kvp_anneal(self._h, C.byref(ap), _ptr(best), C.byref(bt), C.byref(bs), C.byref(stats),
                               _stream(stream)), "kvp_anneal")
        return dict(best_schedule=best, best_ticks=int(bt.value), best_seconds=float(bs.value), stats=stats,
                    per_chain=list(per) if per is not None else None)

    def anneal_exchange(self, ap, rungs, every, want_schedule=True, stream=None):
        """kvp_anneal_exchange -> dict(best_schedule, best_ticks, best_seconds, stats, per_chain, final_rung, n_exchanged)."""
        best = torch.empty((self.steps, self.w32), dtype=torch.int32, device="cuda") if want_schedule else None
        bt = C.c_uint64(); bs = C.c_double()
        stats = AnnealStats()
        per = (ChainResult * ap.chains)()
        stats.per_chain = C.cast(per, C.POINTER(ChainResult))
        final_rung = (C.c_uint32 * ap.chains)()
        n_ex = (C.c_uint32 * ap.chains)()
        xp = ExchangeParams(int(rungs), 0, int(every))
        _chk(_lib().kvp_anneal_exchange(self._h, C.byref(ap), C.byref(xp), _ptr(best), C.byref(bt), C.byref(bs),
                                        C.byref(stats), final_rung, n_ex, _stream(stream)), "kvp_anneal_exchange")
        return dict(best_schedule=best, best_ticks=int(bt.value), best_seconds=float(bs.value), stats=stats,
                    per_chain=list(per), final_rung=list(final_rung), n_exchanged=list(n_ex))

    def chain_state(self, ap, chain, upto_moves, stream=None):
        """kvp_anneal_chain_state -> (schedule CUDA int32 [S][W32], ChainResult)."""
        sched = torch.empty((self.steps, self.w32), dtype=torch.int32, device="cuda")
        res = ChainResult()
        _chk(_lib().kvp_anneal_chain_state(self._h, C.byref(ap), C.c_uint32(chain), C.c_uint64(upto_moves),
                                           _ptr(sched, torch.int32), C.byref(res), _stream(stream)),
             "kvp_anneal_chain_state")
        return sched, res

    def policy_lookahead(self, windows, ratios_permille, init_mode=INIT_STATIC_FIRST, stream=None):
        """kvp_policy_lookahead -> CUDA int32 [n][S][W32], one schedule per (W, R) pair."""
        n = len(windows)
        w = (C.c_uint32 * n)(*[int(x) for x in windows])
        r = (C.c_uint32 * n)(*[int(x) for x in ratios_permille])
        out = torch.empty((n, self.steps, self.w32), dtype=torch.int32, device="cuda")
        _chk(_lib().kvp_policy_lookahead(self._h, C.c_uint32(init_mode), w, r, C.c_uint32(n), _ptr(out), _stream(stream)),
             "kvp_policy_lookahead")
        return out

    def policy_reactive(self, init_mode=INIT_STATIC_FIRST, stream=None):
        """kvp_policy_reactive -> CUDA int32 [S][W32]."""
        out = torch.empty((self.steps, self.w32), dtype=torch.int32, device="cuda")
        _chk(_lib().kvp_policy_reactive(self._h, C.c_uint32(init_mode), _ptr(out), _stream(stream)), "kvp_policy_reactive")
        return out

    def policy_page(self, page_units, stream=None):
        """kvp_policy_page -> CUDA int32 [S][W32]."""
        out = torch.empty((self.steps, self.w32), dtype=torch.int32, device="cuda")
        _chk(_lib().kvp_policy_page(self._h, C.c_uint32(page_units), _ptr(out), _stream(stream)), "kvp_policy_page")
        return out

    def wr_grid(self, w_max, n_ratio=11, init_mode=INIT_STATIC_FIRST, stream=None):
        """kvp_wr_grid -> CUDA int64 [w_max][n_ratio]: total ticks of the look-ahead policy on the (W, R) grid."""
        table = torch.empty((w_max, n_ratio), dtype=torch.int64, device="cuda")
        _chk(_lib().kvp_wr_grid(self._h, C.c_uint32(init_mode), C.c_uint32(w_max), C.c_uint32(n_ratio), _ptr(table),
                                _stream(stream)), "kvp_wr_grid")
        return table


def wr_params(chains, iters, seed=0, levels=16, p0=0.8, alpha=0.9, early_stop_permille=0, w0=1, r0=0):
    wp = WRParams()
    wp.chains, wp.levels, wp.iters, wp.seed = chains, levels, iters, seed
    wp.p0, wp.alpha, wp.early_stop_permille, wp.w0, wp.r0 = p0, alpha, early_stop_permille, w0, r0
    return wp


def wr_anneal(table, wp, stream=None):
    """kvp_wr_anneal on a CUDA int64 table [w_max][n_ratio] -> (list of WRResult per chain, best WRResult)."""
    res = (WRResult * wp.chains)()
    best = WRResult()
    _chk(_lib().kvp_wr_anneal(_ptr(table, torch.int64), C.c_uint32(table.shape[0]), C.c_uint32(table.shape[1]),
                              C.byref(wp), res, C.byref(best), _stream(stream)), "kvp_wr_anneal")
    return list(res), best
