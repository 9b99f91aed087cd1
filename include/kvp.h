/*
 * kvp.h -- C ABI of libkvp: KV-cache placement bound search on one NVIDIA B200.
 *
 * The library scores and searches placement schedules for the problem posed in
 * "Accelerating LLM Inference via Dynamic KV Cache Placement in Heterogeneous
 * Memory System" (arXiv 2508.13231), Section III:
 *
 *   - a KV cache of `units` equally sized blocks, `steps` decode steps, and for
 *     every step the set of blocks that sparse attention reads (access bitmap);
 *   - a placement schedule P: for every step the set of blocks that are resident
 *     in HBM while that step reads (all other blocks are in off-package DRAM);
 *   - the latency model of Eq. 1-4 and the capacity constraint of Eq. 5.
 *
 * Conventions shared by every call
 * --------------------------------
 * Bitmaps. A bitmap has `steps` rows of W32 = ceil(units/32) uint32 words,
 *   row-major ("step-major"). Unit u of step s is bit (u & 31) of word
 *   [s*W32 + (u >> 5)]. Pad bits (u >= units) of the last word are ignored on
 *   input and written as 0 on output.
 * Time. All costs are exact integers ("ticks"). With g = gcd(B_h, B_k, B_d),
 *   B'_x = B_x / g and L = lcm(B'_h, B'_k, B'_d), the weights are
 *   kappa_h = L/B'_h, kappa_k = L/B'_k, kappa_d = L/B'_d,
 *   kappa_e = max(kappa_k, kappa_d)  (the 1/min{B_k,B_d} of Eq. 4),
 *   and one tick lasts bytes_per_unit / (L*g) seconds.
 * Step cost (Eq. 2-4) for step s with previous row P[s-1] (P[-1] := P[0]):
 *   hr = |A[s] & P[s]|, er = |A[s]| - hr, mi = |P[s] & ~P[s-1]|,
 *   mo = |~P[s] & P[s-1]|, Fh/Fe = 1 when KVP_MIG_HBM/KVP_MIG_EXT is set,
 *   th = kappa_h*(hr + hw[s] + Fh*(mi+mo))                              (Eq. 3)
 *   te = kappa_e*er + max(kappa_k*(ew[s] + Fe*mo), kappa_k*Fe*mi,
 *                         kappa_d*(ew[s] + Fe*(mi+mo)))                 (Eq. 4)
 *   f_s = max(th, te)  (Eq. 2);   T = sum_s f_s  (Eq. 1);
 *   feasible iff |P[s]| <= hbm_capacity_units for every s  (Eq. 5).
 * Pointers. Every pointer argument is marked (host) or (device). Device
 *   buffers are owned by the caller, must be 16-byte aligned and must stay
 *   valid until the work queued on `stream` has finished. `stream` is a
 *   cudaStream_t passed as void* (NULL = the legacy default stream).
 * Errors. Every function returns KVP_OK or a negative code; there are no
 *   exceptions, no abort, no output on stdout. On error, outputs are
 *   unspecified but no memory outside the documented buffers is touched.
 *   There is no CPU fallback: without a usable CUDA device every compute
 *   call returns KVP_ERR_CUDA.
 */
#ifndef KVP_H_
#define KVP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KVP_OK             0
#define KVP_ERR_ARG       -1  /* null pointer, zero size, cap > units, bad enum, ...           */
#define KVP_ERR_CAPACITY  -2  /* an initial schedule violates Eq. 5                              */
#define KVP_ERR_RANGE     -3  /* tick weights or sizes outside the supported integer ranges     */
#define KVP_ERR_CUDA      -4  /* a CUDA runtime call failed (see kvp_last_cuda_error)           */
#define KVP_ERR_NOMEM     -5  /* device or host allocation failed                                */
#define KVP_ERR_TIMEOUT   -6  /* a bounded device-side wait expired                              */
#define KVP_ERR_INTERNAL  -7  /* self-check failed: re-scored winner differs from tracked ticks */

#define KVP_MIG_HBM 1u  /* migrations occupy HBM bandwidth: the |M^i|+|M^o| terms of Eq. 3   */
#define KVP_MIG_EXT 2u  /* migrations occupy link/DRAM bandwidth: the M terms of Eq. 4      */
#define KVP_MIG_PAPER (KVP_MIG_HBM | KVP_MIG_EXT)

/* Bandwidths of Eq. 3-4 in bytes per second (Table I gives 4.9e12 / 9e11 / 5e11). */
typedef struct {
    uint64_t bw_hbm;    /* B_h */
    uint64_t bw_link;   /* B_k, uni-directional bandwidth of the full-duplex link */
    uint64_t bw_dram;   /* B_d, off-package DRAM channel bandwidth */
    uint32_t mig_flags; /* KVP_MIG_*; 0 = migrations are free (test mode with a closed-form optimum) */
    uint32_t reserved;  /* must be 0 */
} kvp_memsys;

typedef struct kvp_problem kvp_problem; /* opaque; owns device copies of everything it needs */

/* Derived integer weights of a problem (see "Time" above). */
typedef struct {
    uint64_t kappa_h, kappa_k, kappa_d, kappa_e;
    uint64_t lcm, gcd;
    double   seconds_per_tick;
    uint32_t units, steps, words_per_row, capacity;
} kvp_info;

/*
 * kvp_create -- build a problem instance (Section III-A: units, access pattern
 * known a priori, capacity P_H <= 100% of `hbm_capacity_units`, bandwidths).
 *   out              (host)   receives the handle.
 *   access_bitmaps   (device) [steps][W32], copied; the caller may free it after
 *                             the stream work finished.
 *   hw_units/ew_units (host)  [steps] or NULL (= all zero): |H^w|, |E^w| of
 *                             Eq. 3-4 in units, caller-supplied constants.
 * Limits: 1 <= units < 2^26, 1 <= steps <= 32768, hbm_capacity_units <= units,
 * kappa_max * (2*units + max hw + max ew) < 2^31 (else KVP_ERR_RANGE).
 * Synchronises `stream` before returning.
 */
int kvp_create(kvp_problem** out, uint32_t units, uint64_t bytes_per_unit, uint32_t steps,
               const uint32_t* access_bitmaps, uint32_t hbm_capacity_units,
               const kvp_memsys* mem, const uint32_t* hw_units, const uint32_t* ew_units,
               void* stream);

/* Frees the handle and every device buffer it owns, in stream order behind the last call made on the
 * problem (that stream must still exist). NULL is allowed. Device memory comes from CUDA's stream-ordered
 * allocator. Process-wide side effect: the library raises the release threshold of the device's default memory
 * pool to the largest block it has asked for on that device so far plus 1 GiB (about 42 GB after an annealing
 * call on a 2.6M-unit x 64-step problem), so that the next problem of the same size gets its workspace back
 * without a trip to the driver; the pool keeps that much freed memory after kvp_destroy, where other users of
 * cudaMalloc in the process cannot see it until the pool is trimmed (cudaMemPoolTrimTo). */
void kvp_destroy(kvp_problem* p);

/* Fills *info (host). */
int kvp_get_info(const kvp_problem* p, kvp_info* info);

/*
 * kvp_eval -- score `n` schedules with Eq. 1-4 and test Eq. 5.
 *   schedules     (device) [n][steps][W32]
 *   step_ticks    (device) [n][steps] uint64 or NULL : f_s
 *   total_ticks   (device) [n] uint64                : T
 *   step_seconds  (device) [n][steps] double or NULL : f_s * seconds_per_tick
 *   total_seconds (device) [n] double or NULL        : T * seconds_per_tick
 *   bad_step      (device) [n] int32 or NULL : first step whose row holds more
 *                 than hbm_capacity_units units, or -1 when the schedule is feasible
 *                 (an infeasible schedule is still scored).
 * Asynchronous on `stream`; uses scratch owned by the problem, so calls on the
 * same problem must be issued on one stream at a time.
 */
int kvp_eval(kvp_problem* p, const uint32_t* schedules, uint32_t n,
             uint64_t* step_ticks, uint64_t* total_ticks,
             double* step_seconds, double* total_seconds, int32_t* bad_step, void* stream);

/*
 * kvp_eval_counts -- the four per-step cardinalities the cost model is built on.
 *   counts (device) [n][steps][4] uint32 = {hr, mi, mo, occ} with occ = |P[s]|.
 */
int kvp_eval_counts(kvp_problem* p, const uint32_t* schedules, uint32_t n,
                    uint32_t* counts, void* stream);

/*
 * kvp_eval_noalloc -- kvp_eval for callers that must not allocate device memory. (The paper has no
 * counterpart; this is a service of this library.)
 *
 * kvp_eval keeps its per-step cardinalities in a scratch buffer that it re-allocates whenever a batch is
 * larger than any before. That is unwelcome in three situations: inside a serving or
 * control loop where an allocation would stall the whole device for a moment; in a process whose
 * framework has claimed all device memory for its own pool, so that a raw cudaMalloc fails; and in code
 * that is not allowed to call the allocator at all at that point. This variant takes the same arguments
 * and gives the same results, but its scratch is a fixed array that is part of the library image:
 * KVP_NOALLOC_SCRATCH_BYTES (1 MiB) of device memory on every GPU that loads the library, held until the
 * process exits. It calls no allocating routine, neither of CUDA nor of any other library.
 *
 * Limit: n * steps * 16 bytes <= KVP_NOALLOC_SCRATCH_BYTES, i.e. n * steps <= 65536; a larger batch is
 * refused with KVP_ERR_RANGE and nothing is launched (split it, or use kvp_eval). Every batch inside the limit is
 * served, also the 32,769 to 65,536 one- or two-step schedules that need more than one launch.
 * First call on a device: looks up the device address of the array (once per device, with that device
 * current). Make that first call outside any stream capture.
 * Sharing: every call on a device uses the same array and overwrites what the previous call left there
 * (everything that must start from zero is cleared by the call itself). Two calls whose kernels can
 * overlap on the GPU -- different streams, or different host threads -- race on it; order them.
 * Otherwise as kvp_eval: asynchronous on `stream`, all pointers (device), `p` from kvp_create.
 */
#define KVP_NOALLOC_SCRATCH_BYTES (1u << 20)
int kvp_eval_noalloc(kvp_problem* p, const uint32_t* schedules, uint32_t n,
                     uint64_t* step_ticks, uint64_t* total_ticks,
                     double* step_seconds, double* total_seconds, int32_t* bad_step, void* stream);

/*
 * kvp_set_births -- make the problem a growing cache: the newly written entries H^w and E^w of the scheduling
 * decision S_(n,l) (Section III-A) become part of the schedule.
 *   birth (device) [units] uint32: 0 = the unit exists before the first step (written by the prefill, outside the
 *   model); b >= 1 = the unit is written during step b, b < steps.
 * Meaning for every later call on `p`:
 *   - before step birth[u] the unit is nowhere: its placement bits there are ignored (by kvp_eval) and never set
 *     (by kvp_anneal, whose moves act only on the steps at which the units they name exist), it does not count
 *     towards Eq. 5, and it must not be accessed (KVP_ERR_ARG otherwise);
 *   - at step b the placement bit decides where the new entry is written: set = HBM, it adds to |H^w_b| of
 *     Eq. 3; clear = off-package DRAM, it adds to |E^w_b| of Eq. 4. Being written is not a migration;
 *   - hw_units / ew_units of kvp_create still add to both sets;
 *   - the static initial placements hold a unit of their row from the step it is written.
 * Call it once, directly after kvp_create. Supported afterwards: kvp_eval, kvp_anneal, kvp_anneal_chain_state,
 * kvp_get_info. kvp_eval_counts, kvp_eval_noalloc, the policies and kvp_wr_grid are defined for fixed populations
 * and return KVP_ERR_ARG. Copies `birth`; synchronises `stream`. Errors: KVP_ERR_ARG (null, called twice, a birth
 * >= steps, an access before birth), KVP_ERR_RANGE (the tick range check of kvp_create with the births added to
 * the written units), KVP_ERR_NOMEM, KVP_ERR_CUDA; on error the problem is unchanged.
 */
int kvp_set_births(kvp_problem* p, const uint32_t* birth, void* stream);

/* Initial placement of a chain. */
#define KVP_INIT_STATIC_FIRST 0u /* units 0..cap-1 at every step: the Static Placement baseline (Section IV-A) */
#define KVP_INIT_STATIC_FREQ  1u /* the cap units with most accesses over all steps (ties: lower index)     */
#define KVP_INIT_USER         2u /* init_schedule */

#define KVP_TABLE_Q 1024u        /* entries per temperature level of the acceptance table */

/*
 * Simulated-annealing parameters (Section III-B: Metropolis rule exp(-dT/C),
 * initial acceptance ratio p0 = 0.8, geometric cooling alpha = 0.9, stop when the
 * best improves by < 0.1% across successive temperature levels or the budget ends).
 * The state that is annealed is the schedule itself: each move either swaps the
 * placement of two units or flips one unit over a run of consecutive steps.
 */
typedef struct {
    uint32_t chains;            /* independent chains, >= 1                                         */
    uint32_t levels;            /* temperature levels, 1..4096; level(m) = min(levels-1, m/(moves/levels)) */
    uint64_t moves;             /* proposals per chain, >= 1                                        */
    uint64_t seed;              /* Philox key                                                       */
    double   p0;                /* target initial acceptance of an average uphill move, in (0,1)    */
    double   alpha;             /* geometric cooling factor, in (0,1]                               */
    const double* temps;        /* (host) [levels] temperatures in ticks, or NULL = derive from p0, alpha */
    uint32_t early_stop_permille;   /* stop a chain at a level boundary when its best improved by less
                                       than this many 1/1000 since the previous boundary; 0 = never    */
    uint32_t early_stop_from_level; /* the rule is not applied at boundaries entering levels below this */
    uint32_t init_mode;         /* KVP_INIT_*                                                        */
    uint32_t p_swap_256;        /* P(swap move) * 256, 0..256; the rest are flip moves              */
    uint32_t max_len_log2;      /* run lengths are min(2^k, 30), k uniform in 0..max_len_log2 (<= 5) */
    uint32_t first_chain;       /* index of the first chain: the call runs chains first_chain ..
                                   first_chain+chains-1, so that a job can be split over GPUs or calls */
    const uint32_t* init_schedule;  /* (device) [steps][W32], only for KVP_INIT_USER                */
} kvp_anneal_params;

/* Per-chain outcome. All fields are exact functions of (problem, params, chain). */
typedef struct {
    uint64_t best_ticks;    /* lowest T the chain visited                                          */
    uint64_t best_move;     /* index of the first move after which T == best_ticks;
                               UINT64_MAX when the initial state was never improved               */
    uint64_t final_ticks;   /* T of the state after the last executed move                         */
    uint64_t moves_done;    /* proposals executed (less than `moves` only after an early stop)     */
    uint64_t n_accepted;    /* proposals that passed the Metropolis test (including no-op moves)   */
    uint64_t n_changed;     /* accepted proposals that changed at least one placement bit          */
    uint64_t n_infeasible;  /* flip proposals rejected because they would violate Eq. 5            */
    uint64_t traj_hash;     /* running hash over (move index, T after move) of every changing move */
} kvp_chain_result;

typedef struct {
    uint64_t init_ticks;        /* T of the initial placement                                      */
    uint64_t best_ticks;        /* the bound: min over chains                                      */
    uint32_t best_chain;        /* lowest chain index that reached it (absolute: includes first_chain) */
    uint32_t levels;            /* number of levels actually used                                  */
    uint64_t best_move;
    uint64_t moves_total;       /* sum of moves_done over chains                                   */
    uint64_t calib_mean_delta;  /* mean positive delta of the calibration proposals (0 if temps given) */
    double   temp0;             /* temperature of level 0 in ticks                                 */
    uint64_t winner_hits, winner_accessed; /* sum_s hr and sum_s |A[s]| of the winner: HBM hit rate */
    float    ms_init, ms_chains, ms_finish;   /* device time of the three phases (CUDA events)     */
    uint32_t kernel_launches;   /* kernels this call launched                                      */
    kvp_chain_result* per_chain; /* (host) [chains] or NULL                                        */
    uint32_t chain_launches;    /* launches of the chain kernel (waves of resident chains)         */
    uint32_t resident_chains;   /* chains per wave                                                 */
    uint32_t wide_kernel;       /* 1: the wide chain kernel ran (many chains), 0: the narrow one   */
    uint32_t reserved;
    /* What the evaluations of the wide kernel amounted to, summed over the chains (0 for the narrow kernel): */
    uint64_t work_again;        /* proposals evaluated a second time after a move was applied in their batch   */
    uint64_t work_listed;       /* evaluations that needed more than the placement bits (a cost evaluation)    */
    uint64_t work_items;        /* (proposal, step) pairs whose step cost (Eq. 2-4) was evaluated              */
    /* kvp_anneal_exchange only: */
    uint64_t exchanges_tried, exchanges_accepted;
    uint32_t exchange_rounds, reserved2;
} kvp_anneal_stats;

/*
 * kvp_accept_table -- the quantised Metropolis thresholds kvp_anneal uses.
 * For level j with temperature C_j (ticks; values below 1 are raised to 1):
 *   shift_j = smallest sh >= 0 with 1024 * 2^sh >= 23 * C_j,
 *   table[j][q] = min(2^32 - 1, floor(2^32 * exp(-((q + 0.5) * 2^shift_j) / C_j))).
 * An uphill move with delta > 0 is accepted iff q = delta >> shift_j < 1024 and
 * the move's 32-bit uniform w satisfies w < table[j][q].
 *   temps  (host) [levels]         table (host) [levels][1024]     shifts (host) [levels]
 * Pure host arithmetic; no device work.
 */
int kvp_accept_table(const double* temps, uint32_t levels, uint32_t* table, uint32_t* shifts);

/*
 * kvp_anneal -- run `chains` independent annealing chains, reduce to the best
 * schedule found (the bound of Section III-B) and re-score it with kvp_eval.
 *   best_schedule (device) [steps][W32] or NULL
 *   best_ticks, best_seconds (host) or NULL
 *   stats (host) or NULL; stats->per_chain must be NULL or a host array [chains]
 *   (entry i belongs to chain first_chain + i)
 * Synchronises `stream` before returning.
 * A job of few chains (at most 8 per SM) is served by two warps per chain that take the chain's batches of 32
 * proposals in turn; a job of many chains by one warp per chain that carries four proposals per lane and keeps the
 * chains' schedules, when they do not fit shared memory, as copy-on-write overlays of the one initial schedule. The
 * results are those of the sequential chain either way. The only device-side wait of the library is a warp's wait
 * for its turn in the two-warp form; it is bounded, and a chain whose wait runs out makes the call return
 * KVP_ERR_TIMEOUT (the outputs are then undefined). The library reads no environment variable; the switches that
 * the test-suite needs are set with kvp_set_test_hooks (end of this header).
 */
int kvp_anneal(kvp_problem* p, const kvp_anneal_params* params, uint32_t* best_schedule,
               uint64_t* best_ticks, double* best_seconds, kvp_anneal_stats* stats, void* stream);

/*
 * kvp_anneal_exchange -- replica exchange (parallel tempering) over the temperature ladder of Section III-B. The
 * paper anneals one chain through falling temperatures; here `rungs` replicas form a ladder, replica r starting on
 * rung r, every replica running at the fixed temperature C_r of the rung it holds, and every `exchange_every` moves
 * neighbouring rungs may exchange (the chains keep their schedules, the rungs change hands). The rule is the
 * standard one for Boltzmann weights exp(-T/C): rungs j (hotter) and j+1 with present costs E_j, E_{j+1} exchange
 * with probability min(1, exp((1/C_j - 1/C_{j+1}) (E_j - E_{j+1}))): always when the colder rung holds the worse
 * schedule (or an equal one), else with exp(-d / C_pair), d = E_j - E_{j+1}, 1/C_pair = 1/C_{j+1} - 1/C_j, through
 * the quantised table of kvp_accept_table at the pair temperatures (kvp_exchange_temps); pairs of equal temperature
 * exchange always.
 *   params: as for kvp_anneal with levels == rungs (the ladder: `temps`, or C_0 from p0 and C_{j+1} = alpha C_j),
 *     chains and first_chain multiples of rungs (chain c belongs to ladder c / rungs, so a job can be split by
 *     ladders over GPUs or calls), early_stop_permille == 0.
 *   Round t = 0, 1, ...: every chain proposes its moves t * exchange_every .. (t + 1) * exchange_every - 1 (up to
 *     `moves`); then, unless the budget is used up, the pairs (j, j+1) with j = t (mod 2) try to exchange. The uniform
 *     of pair j of ladder l in round t is word 3 of Philox4x32-10(counter (t_lo, t_hi, l * rungs + j, 6), key seed).
 *   final_rung  (host) [chains] or NULL: the rung each chain holds at the end
 *   n_exchanged (host) [chains] or NULL: the exchanges each chain took part in
 *   best_schedule, best_ticks, best_seconds, stats: as for kvp_anneal (per-chain results over all rounds).
 * Limits: rungs <= 256; rounds * chains <= 2^30 (the rung history is kept); chains whose schedules do not fit shared
 * memory must all be resident at once (KVP_ERR_RANGE otherwise). Synchronises `stream` before returning.
 */
typedef struct {
    uint32_t rungs;             /* replicas per ladder = temperatures of the ladder, 1..256 */
    uint32_t reserved;          /* must be 0 */
    uint64_t exchange_every;    /* moves between exchange rounds, >= 1 */
} kvp_exchange_params;
int kvp_anneal_exchange(kvp_problem* p, const kvp_anneal_params* params, const kvp_exchange_params* xp,
                        uint32_t* best_schedule, uint64_t* best_ticks, double* best_seconds, kvp_anneal_stats* stats,
                        uint32_t* final_rung, uint32_t* n_exchanged, void* stream);

/* Pair temperatures of a ladder (host arithmetic): 1/pair_temps[j] = 1/temps[j+1] - 1/temps[j] with temperatures below
 * one tick counted as one; always[j] = 1 where the pair exchanges unconditionally (equal temperatures). */
int kvp_exchange_temps(const double* temps, uint32_t rungs, double* pair_temps, uint32_t* always);

/*
 * kvp_anneal_chain_state -- replay one chain for its first `upto_moves` proposals
 * and return the schedule it then holds (trajectories are pure functions of
 * (seed, chain, move index), so this reproduces any state kvp_anneal went through).
 *   schedule (device) [steps][W32];  result (host) or NULL.
 */
int kvp_anneal_chain_state(kvp_problem* p, const kvp_anneal_params* params, uint32_t chain,
                           uint64_t upto_moves, uint32_t* schedule, kvp_chain_result* result,
                           void* stream);

/*
 * Synthetic access traces: the stand-in for recorded attention scores
 * (Section IV-A) in the spirit of the synthesised low/high-variation traces of
 * Section IV-B. Units are arranged as `groups` (layer, kv-head) pairs of
 * `units_per_group` blocks; every step each group reads its `topk` most
 * important blocks. Importance of unit u at step t is the integer (Q16.16)
 *   score = x_t(u) + base[u],  x_0 = (sigma_q*e_0) >> 16,
 *   x_t = (rho_q*x_{t-1} + c_q*e_t) >> 16  [+ burst_jump with probability burst_thr/2^32],
 * where e_t is a unit-variance Irwin-Hall(8) variate built from the eight 16-bit
 * halves of Philox4x32-10(counter = (u, t, 0, 3), key = seed):
 *   e = ((sum of halves - 262140) * 80265) >> 16.
 * Ties are broken towards the lower unit index.
 *
 * layers = L > 1: the steps are the (token n, layer l) pairs of Section III-A in the order s = n*L + l. The groups
 * are split into L consecutive blocks of groups/L, one per layer; a group reads only at the steps of its layer
 * (its bits are 0 elsewhere) and the importance of its units advances once per token: the noise counter is
 * (u, n, 0, 3) and x_n follows x_{n-1}. groups must be a multiple of L.
 * birth != NULL (growing cache, see kvp_set_births): at step s a group reads its min(topk, existing) most
 * important existing units, a unit existing from step birth[u] on.
 */
typedef struct {
    uint32_t groups, units_per_group, steps, topk;
    uint64_t seed;
    int32_t  rho_q;       /* AR(1) coefficient * 2^16, 0..65536                      */
    int32_t  c_q;         /* innovation scale * 2^16, 0..2^20                        */
    int32_t  sigma_q;     /* std of x_0 * 2^16, 0..2^20                              */
    int32_t  burst_jump;  /* Q16.16 jump added to x_t when a burst fires             */
    uint32_t burst_thr;   /* burst probability * 2^32 (0 = no bursts)                */
    uint32_t flags;       /* KVP_TRACE_*                                             */
    const int32_t* base;  /* (device) [groups*units_per_group] static log-importance, or NULL = 0;
                             |base| <= 2^29                                          */
    uint32_t layers;      /* 0 or 1: every group reads at every step                 */
    uint32_t reserved;    /* must be 0                                               */
    const uint32_t* birth;/* (device) [groups*units_per_group] or NULL               */
} kvp_trace_params;

#define KVP_TRACE_SINGLE_PASS 1u /* never allocate the [steps][units] int32 score matrix. By default every trace whose
                                    matrix is at most 1 GiB, and that is neither layered nor growing, is generated in
                                    two passes through such a matrix (stream-ordered scratch, freed on return); the
                                    single-pass form is slower, much slower for few groups */

/*
 * kvp_trace_generate -- fill access_bitmaps (device) [steps][ceil(U/32)] with the
 * top-k sets described above. Asynchronous on `stream`.
 * Limits: units_per_group <= 8192, 1 <= topk <= units_per_group (KVP_ERR_RANGE / KVP_ERR_ARG otherwise).
 */
int kvp_trace_generate(const kvp_trace_params* params, uint32_t* access_bitmaps, void* stream);

/*
 * The look-ahead placement policy that the paper's annealer tunes (Section III-B), as a schedule generator.
 * Window W (steps, 1..64) and migration ratio R = ratio_permille / 1000. Starting from the static placement
 * `init_mode` (KVP_INIT_STATIC_FIRST or KVP_INIT_STATIC_FREQ), before every step s:
 *   - the frequency of a unit is the number of its accesses in steps s .. s+W-1;
 *   - candidates are the units outside HBM with frequency > 0, ranked by frequency (ties: lower index); only the
 *     best floor(R * candidates) may migrate;
 *   - they first take free HBM capacity; then the j-th remaining candidate replaces the j-th resident in order of
 *     rising frequency (ties: lower index) as long as that resident is accessed less often than the candidate.
 * The placement decided before step s is the one step s reads (row s of the schedule); the cost model charges the
 * migrations to step s (none at s = 0).
 *   windows, ratios_permille (host) [n];  schedules (device) [n][steps][W32]: one schedule per (W, R) pair.
 * Limit: units <= 32768 (KVP_ERR_RANGE). Synchronises `stream` before returning.
 */
int kvp_policy_lookahead(kvp_problem* p, uint32_t init_mode, const uint32_t* windows,
                         const uint32_t* ratios_permille, uint32_t n, uint32_t* schedules, void* stream);

/*
 * Reactive Scheduling (Section IV-A) as a schedule generator: a unit read while it is outside HBM is promoted, the
 * least recently used resident makes room. The miss of step s is served off-package; the unit is resident from
 * step s+1. Per step the hit units become most recently used; the missed units, in index order and at most
 * `capacity` of them, first take free capacity and then replace residents in order of (last use, index).
 *   schedule (device) [steps][W32]. Limit: units <= 32768. Asynchronous on `stream`.
 */
int kvp_policy_reactive(kvp_problem* p, uint32_t init_mode, uint32_t* schedule, void* stream);

/*
 * Page Granularity Scheduling (Section IV-A) as a schedule generator: placement in pages of page_units consecutive
 * units (a power of two, 2..32, dividing `units`; the paper uses pages of 16 tokens) with perfect foresight of the
 * current step. Before step s a page's score is the number of its units that step s reads; non-resident pages with
 * a positive score, ranked by score (ties: lower index), first take free page slots (floor(capacity / page_units)
 * pages), then the j-th remaining one replaces the j-th resident page in order of rising score while that score is
 * lower. Initial placement: the first pages up to capacity.
 *   schedule (device) [steps][W32]. Limit: units <= 32768. Asynchronous on `stream`.
 */
int kvp_policy_page(kvp_problem* p, uint32_t page_units, uint32_t* schedule, void* stream);

/*
 * kvp_wr_grid -- T(W, R) of the look-ahead policy on the whole grid W = 1..w_max, R = r / (n_ratio - 1),
 * r = 0..n_ratio-1: runs kvp_policy_lookahead and kvp_eval on every grid point.
 *   table (device) [w_max][n_ratio] uint64 total ticks.
 */
int kvp_wr_grid(kvp_problem* p, uint32_t init_mode, uint32_t w_max, uint32_t n_ratio, uint64_t* table, void* stream);

/*
 * The paper's own annealer (Section III-B): state (W, R), objective T(W, R) from a kvp_wr_grid table. Each
 * iteration draws one of three operators with probabilities (0.4, 0.4, 0.2): a window move (W +- 1 or 2), a ratio
 * move (R +- one grid step, 0.1 for n_ratio = 11), or both at once; a proposal that leaves the grid is discarded.
 * Metropolis acceptance exp(-dT/C) with the quantised table of kvp_accept_table; C_0 accepts the mean uphill step
 * between grid neighbours with probability p0 and C_{j+1} = alpha * C_j over `levels` levels of iters/levels
 * iterations; with early_stop_permille a chain stops at a level boundary when its best improved by less than that
 * many 1/1000 since the previous boundary. Iteration i of chain c uses Philox4x32-10(counter (i_lo, i_hi, c, 5), key
 * seed): operator from the low byte of word 0 (< 102: window, < 204: ratio, else both), the W step from bits 8-9
 * ({-2, -1, +1, +2}), the R direction from bit 10, the Metropolis uniform is word 3.
 */
typedef struct {
    uint32_t chains, levels;
    uint64_t iters, seed;
    double   p0, alpha;             /* the paper: 0.8, 0.9 */
    uint32_t early_stop_permille;   /* the paper: 1 (0.1%); 0 = never */
    uint32_t w0, r0;                /* start: W = w0 (1..w_max), R = r0 / (n_ratio - 1) */
    uint32_t reserved;              /* must be 0 */
} kvp_wr_params;

typedef struct {
    uint64_t best_ticks, final_ticks, iters_done, n_accepted;
    uint32_t best_w, best_r, final_w, final_r;
} kvp_wr_result;

/*
 * kvp_wr_anneal -- run `chains` independent (W, R) chains on a table.
 *   table (device) [w_max][n_ratio];  results (host) [chains] or NULL;  best (host) or NULL: the chain with the
 *   lowest best_ticks (ties: lower chain index). Synchronises `stream`.
 */
int kvp_wr_anneal(const uint64_t* table, uint32_t w_max, uint32_t n_ratio, const kvp_wr_params* params,
                  kvp_wr_result* results, kvp_wr_result* best, void* stream);

/* Philox4x32-10 (Salmon et al., SC'11) on the host; exposed so that callers can
 * reproduce which proposal a given (seed, chain, move) pair is. */
void kvp_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);

/*
 * ---- test only ----
 * Switches of the test-suite (and of tuning runs); process-wide, read at the start of every kvp_anneal /
 * kvp_anneal_chain_state. No production caller needs them. All zero = the library's normal behaviour; NULL resets.
 */
typedef struct {
    uint32_t warps_per_chain;   /* 1 or 2: the narrow chain kernel with that many warps per chain; 3: the wide
                                   chain kernel (one warp, four proposals per lane); whatever the job size       */
    uint32_t drop_turn;         /* 1: withhold one hand-over per chain so that the bounded wait for the turn
                                   runs out (about a second) and the call returns KVP_ERR_TIMEOUT               */
    uint32_t split_queue_plus1; /* n + 1: batches with more than n work items take the rarely reached two-halves
                                   path of the half-size work queue                                              */
    uint32_t resident;          /* n: at most n chains whose schedules live in global memory run at a time, so
                                   that a small job comes in several waves                                       */
    uint32_t overlay;           /* narrow chain kernel, schedules in global memory: 1 = copy-on-write slices, 2 =
                                   plain slices, whatever the size of the job (0: by size)                       */
} kvp_test_hooks;
void kvp_set_test_hooks(const kvp_test_hooks* hooks);

const char* kvp_strerror(int code);
/* Text of the last CUDA error seen by the calling thread ("" if none). */
const char* kvp_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* KVP_H_ */
