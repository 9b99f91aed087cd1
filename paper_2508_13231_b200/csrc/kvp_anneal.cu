// Annealing kernels: one chain per warp, lanes spread over the steps a proposal touches.
//
// State of a chain: the schedule in time-packed form (for every unit a bit string over the steps), either
// in shared memory (small problems) or in a private slice of global scratch, plus the four per-step
// cardinalities {hr, mi, mo, occ} in shared memory and the running total T in registers.
//
// A proposal (one Philox4x32-10 block, a pure function of seed, chain and move index) names a run of at most
// 31 consecutive steps and one or two units. Only the run's steps and the step after it change cost, so
// lane j re-evaluates step s0 + j with Eq. 2-4 from the counters and a handful of bit reads, the warp sums
// the differences with one redux, and one thread-uniform Metropolis test against the quantised
// exp(-delta/C) table decides. Philox blocks are drawn 32 moves at a time, one per lane.
#include <math.h>
#include <string.h>

#include <vector>

#include "kvp_common.cuh"

namespace kvp {

namespace {

struct ChainParams {
    const uint32_t* Acol;        // [U][S32]
    const StepC* stepc;          // [S]
    const uint4* counters0;      // [S] counters of the initial schedule
    const uint32_t* Pcol0;       // [U][S32] initial schedule
    const uint32_t* table;       // [levels][1024]
    const uint32_t* shifts;      // [levels]
    uint32_t* ws;                // global scratch: [slots][U*S32] (only the global-state variant)
    kvp_chain_result* results;   // indexed by chain - result_base
    uint32_t* dump;              // if set, slot 0 writes its final schedule here (time-packed)
    CostK K;
    uint32_t U, S, S32, cap;
    uint32_t chain_first, chain_count, result_base;
    uint32_t levels, p_swap_256, len_choices;
    uint32_t early_permille, early_from;
    uint32_t seed_lo, seed_hi;
    uint64_t per_level, upto, init_ticks;
};

// What a lane needs to remember between evaluating and applying a proposal.
struct LaneDelta {
    uint4 ctr;                   // counters of the lane's step before the move
    int dhr, dmi, dmo, docc;
    uint32_t t;                  // the lane's step (valid when active)
    bool active;
};

__device__ __forceinline__ void decode_move(const uint32_t r[4], uint32_t p_swap_256, uint32_t len_choices, uint32_t S,
                                            uint32_t U, uint32_t& pk, uint32_t& u, uint32_t& v)
{
    const uint32_t swap = (r[0] & 255u) < p_swap_256 ? 1u : 0u;
    const uint32_t k = (((r[0] >> 8) & 255u) * len_choices) >> 8;
    const uint32_t len = min(1u << k, 31u);
    const uint32_t s0 = ((r[0] >> 16) * S) >> 16;
    pk = swap | (len << 1) | (s0 << 8);
    u = __umulhi(r[1], U);
    v = __umulhi(r[2], U);
}

// Evaluate a proposal against the current state. All 32 lanes call this with identical arguments.
// Returns the summed cost change; `infeasible` (a flip would break Eq. 5) and `changed` are warp-uniform.
template <typename CtrPtr>
__device__ __forceinline__ int eval_move(const uint32_t* P, const uint32_t* __restrict__ Acol, CtrPtr ctr,
                                         const StepC* __restrict__ stepc, const CostK K, uint32_t S, uint32_t S32,
                                         uint32_t cap, uint32_t lane, uint32_t pk, uint32_t u, uint32_t v,
                                         LaneDelta& ld, bool& infeasible, bool& changed)
{
    const bool swap = pk & 1u;
    const uint32_t len = (pk >> 1) & 63u, s0 = pk >> 8;
    const uint32_t last = min(s0 + len, S - 1);
    const uint32_t t = s0 + lane;
    const bool active = t <= last;
    const uint32_t tt = active ? t : s0;
    const bool in_run = active && lane < len;                      // the placement bit of step t changes hands
    const bool prev_in_run = active && (tt == 0 ? in_run : lane >= 1);  // step 0 has no predecessor: P[-1] := P[0]
    const uint32_t tp = tt ? tt - 1 : 0;
    const size_t ub = (size_t)u * S32, vb = (size_t)v * S32;
    const uint32_t wi = tt >> 5, bi = tt & 31, wpi = tp >> 5, bpi = tp & 31;

    const uint32_t pu = (P[ub + wi] >> bi) & 1u, qu = (P[ub + wpi] >> bpi) & 1u;
    const uint32_t au = (__ldg(Acol + ub + wi) >> bi) & 1u;
    uint32_t pv = 0, qv = 0, av = 0;
    if (swap) {
        pv = (P[vb + wi] >> bi) & 1u; qv = (P[vb + wpi] >> bpi) & 1u;
        av = (__ldg(Acol + vb + wi) >> bi) & 1u;
    }
    uint32_t npu, nqu, npv, nqv;
    if (swap) {
        npu = in_run ? pv : pu; npv = in_run ? pu : pv;
        nqu = prev_in_run ? qv : qu; nqv = prev_in_run ? qu : qv;
    } else {
        npu = pu ^ (in_run ? 1u : 0u); nqu = qu ^ (prev_in_run ? 1u : 0u);
        npv = 0; nqv = 0;
    }
    ld.dhr = (int)(au & npu) - (int)(au & pu) + (int)(av & npv) - (int)(av & pv);
    ld.dmi = (int)(npu & ~nqu & 1u) - (int)(pu & ~qu & 1u) + (int)(npv & ~nqv & 1u) - (int)(pv & ~qv & 1u);
    ld.dmo = (int)(~npu & nqu & 1u) - (int)(~pu & qu & 1u) + (int)(~npv & nqv & 1u) - (int)(~pv & qv & 1u);
    ld.docc = (int)npu - (int)pu + (int)npv - (int)pv;
    ld.active = active;
    ld.t = tt;
    ld.ctr = ctr[tt];
    const StepC c = __ldg(stepc + tt);
    const uint32_t f_old = step_cost(ld.ctr.x, ld.ctr.y, ld.ctr.z, c, K);
    const uint32_t f_new = step_cost(ld.ctr.x + ld.dhr, ld.ctr.y + ld.dmi, ld.ctr.z + ld.dmo, c, K);
    const int dl = active ? (int)(f_new - f_old) : 0;
    infeasible = __any_sync(0xFFFFFFFFu, active && ld.docc > 0 && ld.ctr.w + (uint32_t)ld.docc > cap);
    changed = __any_sync(0xFFFFFFFFu, active && (npu != pu || npv != pv));
    return __reduce_add_sync(0xFFFFFFFFu, dl);
}

__device__ __forceinline__ void apply_move(uint32_t* P, uint4* ctr, uint32_t S, uint32_t S32, uint32_t lane,
                                           uint32_t pk, uint32_t u, uint32_t v, const LaneDelta& ld)
{
    const bool swap = pk & 1u;
    const uint32_t len = (pk >> 1) & 63u, s0 = pk >> 8;
    if (ld.active)
        ctr[ld.t] = make_uint4(ld.ctr.x + ld.dhr, ld.ctr.y + ld.dmi, ld.ctr.z + ld.dmo, ld.ctr.w + ld.docc);
    if (lane < 2) {
        const uint32_t end = min(s0 + len, S);
        const uint32_t wj = (s0 >> 5) + lane;
        const uint32_t lo = max(s0, wj * 32u), hi = min(end, wj * 32u + 32u);
        if (hi > lo) {                                   // run lengths are at most 31, so never a full word
            const uint32_t mask = ((1u << (hi - lo)) - 1u) << (lo - wj * 32u);
            const size_t iu = (size_t)u * S32 + wj;
            if (swap) {
                const size_t iv = (size_t)v * S32 + wj;
                const uint32_t a = P[iu], b = P[iv];
                const uint32_t d = (a ^ b) & mask;
                if (d) { P[iu] = a ^ d; P[iv] = b ^ d; }
            } else {
                P[iu] ^= mask;
            }
        }
    }
    __syncwarp();
}

template <bool PSMEM>
__global__ void __launch_bounds__(512)
chain_kernel(const ChainParams prm)
{
    extern __shared__ uint4 smem4[];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = blockDim.x >> 5;
    const uint32_t slot = blockIdx.x * wpb + warp;
    if (slot >= prm.chain_count) return;
    const uint32_t chain = prm.chain_first + slot;
    const uint32_t S = prm.S, S32 = prm.S32, U = prm.U;
    const size_t pwords = (size_t)U * S32;
    uint4* ctr = smem4 + (size_t)warp * S;
    uint32_t* P = PSMEM ? reinterpret_cast<uint32_t*>(smem4 + (size_t)wpb * S) + (size_t)warp * pwords
                        : prm.ws + (size_t)slot * pwords;
    for (uint32_t i = lane; i < S; i += 32) ctr[i] = __ldg(prm.counters0 + i);
    for (size_t i = lane; i < pwords; i += 32) P[i] = __ldg(prm.Pcol0 + i);
    __syncwarp();

    uint64_t cur = prm.init_ticks, best = cur, best_move = ~0ull, best_at_boundary = cur;
    uint64_t n_acc = 0, n_chg = 0, n_inf = 0, hash = 0;
    uint32_t level = 0, shift = __ldg(prm.shifts);
    const uint32_t* trow = prm.table;
    uint64_t next_boundary = prm.levels > 1 ? prm.per_level : ~0ull;
    uint64_t m = 0;
    bool stop = false;
    while (m < prm.upto && !stop) {
        // one Philox block per lane: the proposals of moves m .. m+31
        uint32_t r[4], my_pk, my_u, my_v;
        const uint64_t mine = m + lane;
        philox4x32_10((uint32_t)mine, (uint32_t)(mine >> 32), chain, TAG_MOVE, prm.seed_lo, prm.seed_hi, r);
        decode_move(r, prm.p_swap_256, prm.len_choices, S, U, my_pk, my_u, my_v);
        const uint32_t my_w = r[3];
        const uint32_t nb = (uint32_t)min((uint64_t)32, prm.upto - m);
        for (uint32_t i = 0; i < nb; ++i, ++m) {
            if (m == next_boundary) {                    // a new temperature level starts at this move
                ++level;
                if (prm.early_permille && level >= prm.early_from &&
                    (best_at_boundary - best) * 1000ull < best_at_boundary * (uint64_t)prm.early_permille) {
                    stop = true;
                    break;
                }
                best_at_boundary = best;
                shift = __ldg(prm.shifts + level);
                trow = prm.table + (size_t)level * KVP_TABLE_Q;
                next_boundary = level + 1 < prm.levels ? next_boundary + prm.per_level : ~0ull;
            }
            const uint32_t pk = __shfl_sync(0xFFFFFFFFu, my_pk, i);
            const uint32_t u = __shfl_sync(0xFFFFFFFFu, my_u, i);
            const uint32_t v = __shfl_sync(0xFFFFFFFFu, my_v, i);
            const uint32_t w = __shfl_sync(0xFFFFFFFFu, my_w, i);
            LaneDelta ld;
            bool infeasible, changed;
            const int delta = eval_move(P, prm.Acol, ctr, prm.stepc, prm.K, S, S32, prm.cap, lane, pk, u, v, ld,
                                        infeasible, changed);
            if (infeasible) { ++n_inf; continue; }
            bool accept = delta <= 0;
            if (!accept) {
                const uint32_t q = (uint32_t)delta >> shift;
                accept = q < KVP_TABLE_Q && w < __ldg(trow + q);      // Metropolis, quantised exp(-delta/C)
            }
            if (!accept) continue;
            ++n_acc;
            if (!changed) continue;
            apply_move(P, ctr, S, S32, lane, pk, u, v, ld);
            ++n_chg;
            cur = (uint64_t)((int64_t)cur + delta);
            hash = (hash ^ m) * 0x9E3779B97F4A7C15ull + cur;
            if (cur < best) { best = cur; best_move = m; }
        }
    }
    if (lane == 0) {
        kvp_chain_result res;
        res.best_ticks = best; res.best_move = best_move; res.final_ticks = cur; res.moves_done = m;
        res.n_accepted = n_acc; res.n_changed = n_chg; res.n_infeasible = n_inf; res.traj_hash = hash;
        prm.results[chain - prm.result_base] = res;
    }
    if (prm.dump && slot == 0) {
        __syncwarp();
        for (size_t i = lane; i < pwords; i += 32) prm.dump[i] = P[i];
    }
}

// Calibration of the temperature ladder: proposals (i, 0, 0, TAG_CALIB), i < 1024, are evaluated against the
// initial schedule and never applied; acc = {sum of positive deltas, their number}.
__global__ void __launch_bounds__(256)
calib_kernel(const ChainParams prm, unsigned long long* acc)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= CALIB_N) return;
    uint32_t r[4], pk, u, v;
    philox4x32_10(i, 0u, 0u, TAG_CALIB, prm.seed_lo, prm.seed_hi, r);
    decode_move(r, prm.p_swap_256, prm.len_choices, prm.S, prm.U, pk, u, v);
    LaneDelta ld;
    bool infeasible, changed;
    const int delta = eval_move(prm.Pcol0, prm.Acol, prm.counters0, prm.stepc, prm.K, prm.S, prm.S32, prm.cap, lane,
                                pk, u, v, ld, infeasible, changed);
    if (lane == 0 && !infeasible && delta > 0) {
        atomicAdd(acc, (unsigned long long)delta);
        atomicAdd(acc + 1, 1ull);
    }
}

struct ReduceOut {
    uint64_t best_ticks, best_move, moves_total;
    uint32_t best_chain, pad;
};

// Cross-chain best-so-far: lexicographic minimum of (best_ticks, chain index), plus the executed-move total.
__global__ void __launch_bounds__(1024)
reduce_kernel(const kvp_chain_result* __restrict__ res, uint32_t chains, ReduceOut* out)
{
    __shared__ uint64_t s_t[32], s_m[32];
    __shared__ uint32_t s_c[32];
    uint64_t bt = ~0ull, moves = 0;
    uint32_t bc = 0xFFFFFFFFu;
    for (uint32_t c = threadIdx.x; c < chains; c += blockDim.x) {
        const uint64_t t = res[c].best_ticks;
        moves += res[c].moves_done;
        if (t < bt || (t == bt && c < bc)) { bt = t; bc = c; }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const uint64_t ot = __shfl_xor_sync(0xFFFFFFFFu, bt, off);
        const uint32_t oc = __shfl_xor_sync(0xFFFFFFFFu, bc, off);
        moves += __shfl_xor_sync(0xFFFFFFFFu, moves, off);
        if (ot < bt || (ot == bt && oc < bc)) { bt = ot; bc = oc; }
    }
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { s_t[warp] = bt; s_c[warp] = bc; s_m[warp] = moves; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (uint32_t w = 1; w < (blockDim.x >> 5); ++w) {
            moves += s_m[w];
            if (s_t[w] < bt || (s_t[w] == bt && s_c[w] < bc)) { bt = s_t[w]; bc = s_c[w]; }
        }
        out->best_ticks = bt; out->best_chain = bc; out->moves_total = moves;
        out->best_move = res[bc].best_move;
        out->pad = 0;
    }
}

inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// Everything a run needs on the device, carved out of the problem's chain workspace.
struct Ctx {
    cudaStream_t st;
    ChainParams prm;
    uint32_t* P0;            // [S][W32] initial schedule, step-major
    uint32_t* Pcol0;         // [U][S32]
    uint32_t* counts0;       // [S][4]
    uint64_t* small;         // [0] total ticks, [1] hits, [2] bad step (int32), [4..5] calibration, [8..] reduce out
    uint32_t* table; uint32_t* shifts;
    kvp_chain_result* results;
    uint32_t* dumpcol;       // [U][S32]
    uint32_t* sched;         // [S][W32]
    uint32_t* slots;         // chain state slices (global variant)
    bool psmem;
    uint32_t wpb;            // warps per CTA
    uint32_t resident;       // chains per wave
    size_t smem_per_warp;
    std::vector<double> temps;
    uint64_t init_ticks, calib_mean;
    uint32_t launches;
};

int validate(const kvp_problem* p, const kvp_anneal_params* a)
{
    if (!p || !a) return KVP_ERR_ARG;
    if (!a->chains || !a->moves || !a->levels || a->levels > 4096) return KVP_ERR_ARG;
    if (a->p_swap_256 > 256 || a->max_len_log2 > 5 || a->init_mode > KVP_INIT_USER) return KVP_ERR_ARG;
    if (a->init_mode == KVP_INIT_USER && !a->init_schedule) return KVP_ERR_ARG;
    if (!a->temps && (!(a->p0 > 0.0 && a->p0 < 1.0) || !(a->alpha > 0.0 && a->alpha <= 1.0))) return KVP_ERR_ARG;
    if (a->chains >= (1u << 24) || (uint64_t)a->first_chain + a->chains > (1ull << 31)) return KVP_ERR_RANGE;
    return KVP_OK;
}

template <bool PSMEM>
int launch_chains(const Ctx& c, const ChainParams& prm, uint32_t count)
{
    const uint32_t grid = (count + c.wpb - 1) / c.wpb;
    const size_t smem = (size_t)c.wpb * c.smem_per_warp;
    chain_kernel<PSMEM><<<grid, c.wpb * 32, smem, c.st>>>(prm);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

int run_chains(Ctx& c, uint32_t first, uint32_t count, uint32_t result_base, kvp_chain_result* results, uint64_t upto,
               uint32_t* dump)
{
    ChainParams prm = c.prm;
    prm.chain_first = first; prm.chain_count = count; prm.result_base = result_base;
    prm.results = results; prm.upto = upto; prm.dump = dump;
    ++c.launches;
    return c.psmem ? launch_chains<true>(c, prm, count) : launch_chains<false>(c, prm, count);
}

// Initial schedule, its counters and cost, the temperature ladder and the acceptance table.
int prepare(kvp_problem* p, const kvp_anneal_params* a, cudaStream_t st, Ctx& c)
{
    int rc = validate(p, a);
    if (rc) return rc;
    KVP_CUDA(cudaSetDevice(p->device));
    c.st = st;
    c.launches = 0;
    const size_t sched_bytes = align256((size_t)p->S * p->W32 * 4);
    const size_t col_bytes = align256((size_t)p->U * p->S32 * 4);

    // shared-memory residency of the schedule, else a slice of global scratch per resident chain
    int dev = p->device, smem_max = 0, sms = 0;
    KVP_CUDA(cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    KVP_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const size_t budget = (size_t)smem_max - 1024;
    const size_t ctr_bytes = (size_t)p->S * 16;
    const size_t psmem_per_warp = ctr_bytes + (size_t)p->U * p->S32 * 4;
    c.psmem = psmem_per_warp <= budget / 2;
    if (c.psmem) {
        c.smem_per_warp = psmem_per_warp;
        uint32_t wmax = (uint32_t)(budget / psmem_per_warp);
        if (wmax > 16) wmax = 16;
        uint32_t want = (a->chains + sms - 1) / sms;
        c.wpb = want < 1 ? 1 : (want > wmax ? wmax : want);
        c.resident = a->chains;
        KVP_CUDA(cudaFuncSetAttribute(chain_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)budget));
    } else {
        if (ctr_bytes > budget) return KVP_ERR_RANGE;
        c.smem_per_warp = ctr_bytes;
        uint32_t wmax = (uint32_t)(budget / 2 / ctr_bytes);
        c.wpb = wmax < 1 ? 1 : (wmax > 16 ? 16 : wmax);
        KVP_CUDA(cudaFuncSetAttribute(chain_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)budget));
        int ctas = 0;
        KVP_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&ctas, chain_kernel<false>, (int)c.wpb * 32,
                                                               c.wpb * c.smem_per_warp));
        if (ctas < 1) return KVP_ERR_RANGE;
        uint32_t per_sm = (uint32_t)ctas * c.wpb;                  // resident chains per SM, at most 32
        if (per_sm > 32) per_sm = 32 / c.wpb ? 32 / c.wpb * c.wpb : c.wpb;
        size_t free_b = 0, total_b = 0;
        KVP_CUDA(cudaMemGetInfo(&free_b, &total_b));
        free_b += p->chain_ws_bytes;                               // what we already hold can be reused
        const size_t usable = free_b / 10 * 7;
        size_t fit = usable / col_bytes;
        if (fit < 1) return KVP_ERR_NOMEM;
        size_t cap_r = (size_t)per_sm * sms;
        size_t r = a->chains < cap_r ? a->chains : cap_r;
        if (r > fit) r = fit;
        const uint32_t waves = (uint32_t)((a->chains + r - 1) / r);
        c.resident = (a->chains + waves - 1) / waves;              // equal waves
    }

    // workspace layout
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += align256(bytes); return o; };
    const size_t o_P0 = take(sched_bytes), o_col0 = take(col_bytes), o_cnt = take((size_t)p->S * 16);
    const size_t o_small = take(256), o_table = take((size_t)a->levels * KVP_TABLE_Q * 4), o_shift = take((size_t)a->levels * 4);
    const size_t o_res = take((size_t)(a->chains + 1) * sizeof(kvp_chain_result));
    const size_t o_dump = take(col_bytes), o_sched = take(sched_bytes);
    const size_t o_slots = take(c.psmem ? 0 : (size_t)c.resident * col_bytes);
    rc = ensure_chain_ws(p, off);
    if (rc) return rc;
    char* base = static_cast<char*>(p->d_chain_ws);
    c.P0 = (uint32_t*)(base + o_P0); c.Pcol0 = (uint32_t*)(base + o_col0); c.counts0 = (uint32_t*)(base + o_cnt);
    c.small = (uint64_t*)(base + o_small); c.table = (uint32_t*)(base + o_table); c.shifts = (uint32_t*)(base + o_shift);
    c.results = (kvp_chain_result*)(base + o_res); c.dumpcol = (uint32_t*)(base + o_dump);
    c.sched = (uint32_t*)(base + o_sched); c.slots = (uint32_t*)(base + o_slots);

    // initial schedule in both layouts
    if (a->init_mode == KVP_INIT_USER) {
        if ((rc = launch_clean_copy(a->init_schedule, c.P0, p->S, p->W32, p->pad_mask, st))) return rc;
        if ((rc = launch_bit_transpose(c.P0, p->S, p->W32, p->U, c.Pcol0, p->S32, st))) return rc;
        c.launches += 2;
    } else {
        const uint32_t* row = p->d_row_freq;
        if (a->init_mode == KVP_INIT_STATIC_FIRST) {
            if ((rc = launch_static_first_row(p, c.sched, st))) return rc;
            row = c.sched;
            ++c.launches;
        }
        if ((rc = launch_broadcast_row(row, p->S, p->W32, c.P0, st))) return rc;
        if ((rc = launch_row_to_columns(row, p->U, p->S, p->S32, c.Pcol0, st))) return rc;
        c.launches += 2;
    }
    if ((rc = launch_counts(p, c.P0, 1, c.counts0, st, &c.launches))) return rc;
    if ((rc = launch_finish(p, c.counts0, 1, nullptr, c.small, nullptr, nullptr, (int32_t*)(c.small + 2), c.small + 1, st)))
        return rc;
    ++c.launches;

    ChainParams& prm = c.prm;
    memset(&prm, 0, sizeof prm);
    prm.Acol = p->dAcol; prm.stepc = p->d_stepc; prm.counters0 = (const uint4*)c.counts0; prm.Pcol0 = c.Pcol0;
    prm.table = c.table; prm.shifts = c.shifts; prm.ws = c.slots; prm.K = p->K;
    prm.U = p->U; prm.S = p->S; prm.S32 = p->S32; prm.cap = p->cap;
    prm.levels = a->levels; prm.p_swap_256 = a->p_swap_256; prm.len_choices = a->max_len_log2 + 1;
    prm.early_permille = a->early_stop_permille; prm.early_from = a->early_stop_from_level;
    prm.seed_lo = (uint32_t)a->seed; prm.seed_hi = (uint32_t)(a->seed >> 32);
    prm.per_level = a->moves / a->levels ? a->moves / a->levels : 1;

    // temperature ladder
    c.temps.resize(a->levels);
    c.calib_mean = 0;
    const bool calibrate = a->temps == nullptr;
    if (calibrate) {
        KVP_CUDA(cudaMemsetAsync(c.small + 4, 0, 16, st));
        calib_kernel<<<CALIB_N / 8, 256, 0, st>>>(prm, (unsigned long long*)(c.small + 4));
        KVP_CUDA(cudaGetLastError());
        ++c.launches;
    }
    uint64_t host_small[8];
    KVP_CUDA(cudaMemcpyAsync(host_small, c.small, sizeof host_small, cudaMemcpyDeviceToHost, st));
    KVP_CUDA(cudaStreamSynchronize(st));
    if ((int32_t)(host_small[2] & 0xFFFFFFFFu) >= 0) return KVP_ERR_CAPACITY;   // Eq. 5 on the initial schedule
    c.init_ticks = host_small[0];
    prm.init_ticks = c.init_ticks;
    if (calibrate) {
        uint64_t mean = host_small[5] ? host_small[4] / host_small[5] : 1;
        if (!mean) mean = 1;
        c.calib_mean = mean;
        double C = -(double)mean / log(a->p0);
        for (uint32_t j = 0; j < a->levels; ++j) { c.temps[j] = C; C = C * a->alpha; }
    } else {
        for (uint32_t j = 0; j < a->levels; ++j) c.temps[j] = a->temps[j];
    }
    std::vector<uint32_t> table((size_t)a->levels * KVP_TABLE_Q), shifts(a->levels);
    if ((rc = kvp_accept_table(c.temps.data(), a->levels, table.data(), shifts.data()))) return rc;
    KVP_CUDA(cudaMemcpyAsync(c.table, table.data(), table.size() * 4, cudaMemcpyHostToDevice, st));
    KVP_CUDA(cudaMemcpyAsync(c.shifts, shifts.data(), shifts.size() * 4, cudaMemcpyHostToDevice, st));
    KVP_CUDA(cudaStreamSynchronize(st));           // the host vectors go out of scope
    return KVP_OK;
}

// Replay `chain` for `upto` proposals and leave its schedule, step-major, in c.sched.
int replay_to_sched(kvp_problem* p, Ctx& c, uint32_t chain, uint64_t upto, kvp_chain_result* result_dev)
{
    int rc;
    if (upto == 0) {
        KVP_CUDA(cudaMemcpyAsync(c.sched, c.P0, (size_t)p->S * p->W32 * 4, cudaMemcpyDeviceToDevice, c.st));
        return KVP_OK;
    }
    if ((rc = run_chains(c, chain, 1, chain, result_dev, upto, c.dumpcol))) return rc;
    if ((rc = launch_bit_transpose(c.dumpcol, p->U, p->S32, p->S, c.sched, p->W32, c.st))) return rc;
    ++c.launches;
    return KVP_OK;
}

}  // namespace

}  // namespace kvp

using namespace kvp;

extern "C" int kvp_anneal(kvp_problem* p, const kvp_anneal_params* a, uint32_t* best_schedule, uint64_t* best_ticks,
                          double* best_seconds, kvp_anneal_stats* stats, void* stream)
{
    Ctx c;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc = validate(p, a);
    if (rc) return rc;
    KVP_CUDA(cudaSetDevice(p->device));
    cudaEvent_t ev[4];
    for (auto& e : ev) KVP_CUDA(cudaEventCreate(&e));
    auto cleanup = [&]() { for (auto& e : ev) cudaEventDestroy(e); };
    KVP_CUDA(cudaEventRecord(ev[0], st));
    if ((rc = prepare(p, a, st, c))) { cleanup(); return rc; }
    KVP_CUDA(cudaEventRecord(ev[1], st));

    // the chains, one wave of resident chains after the other
    for (uint32_t first = 0; first < a->chains; first += c.resident) {
        const uint32_t count = a->chains - first < c.resident ? a->chains - first : c.resident;
        if ((rc = run_chains(c, a->first_chain + first, count, a->first_chain, c.results, a->moves, nullptr))) {
            cleanup(); return rc;
        }
    }
    KVP_CUDA(cudaEventRecord(ev[2], st));

    // cross-chain reduction, then the winner's schedule by deterministic replay and a re-score
    ReduceOut* red_dev = reinterpret_cast<ReduceOut*>(c.small + 8);
    reduce_kernel<<<1, 1024, 0, st>>>(c.results, a->chains, red_dev);
    KVP_CUDA(cudaGetLastError());
    ++c.launches;
    ReduceOut red;
    KVP_CUDA(cudaMemcpyAsync(&red, red_dev, sizeof red, cudaMemcpyDeviceToHost, st));
    KVP_CUDA(cudaStreamSynchronize(st));
    const uint64_t upto = red.best_move == ~0ull ? 0 : red.best_move + 1;
    red.best_chain += a->first_chain;                      // the reduction works on call-local indices
    if ((rc = replay_to_sched(p, c, red.best_chain, upto, c.results + a->chains))) { cleanup(); return rc; }
    if ((rc = launch_counts(p, c.sched, 1, c.counts0, st, &c.launches))) { cleanup(); return rc; }
    if ((rc = launch_finish(p, c.counts0, 1, nullptr, c.small, nullptr, nullptr, (int32_t*)(c.small + 2), c.small + 1, st))) {
        cleanup(); return rc;
    }
    ++c.launches;
    if (best_schedule)
        KVP_CUDA(cudaMemcpyAsync(best_schedule, c.sched, (size_t)p->S * p->W32 * 4, cudaMemcpyDeviceToDevice, st));
    uint64_t host_small[4];
    KVP_CUDA(cudaMemcpyAsync(host_small, c.small, sizeof host_small, cudaMemcpyDeviceToHost, st));
    if (stats && stats->per_chain)
        KVP_CUDA(cudaMemcpyAsync(stats->per_chain, c.results, (size_t)a->chains * sizeof(kvp_chain_result),
                                 cudaMemcpyDeviceToHost, st));
    KVP_CUDA(cudaEventRecord(ev[3], st));
    KVP_CUDA(cudaStreamSynchronize(st));
    const bool ok = host_small[0] == red.best_ticks && (int32_t)(host_small[2] & 0xFFFFFFFFu) < 0;
    if (best_ticks) *best_ticks = red.best_ticks;
    if (best_seconds) *best_seconds = (double)red.best_ticks * p->spt;
    if (stats) {
        kvp_chain_result* keep = stats->per_chain;
        memset(stats, 0, sizeof *stats);
        stats->per_chain = keep;
        stats->init_ticks = c.init_ticks; stats->best_ticks = red.best_ticks; stats->best_chain = red.best_chain;
        stats->levels = a->levels; stats->best_move = red.best_move; stats->moves_total = red.moves_total;
        stats->calib_mean_delta = c.calib_mean; stats->temp0 = c.temps[0];
        stats->winner_hits = host_small[1]; stats->winner_accessed = p->total_accessed;
        cudaEventElapsedTime(&stats->ms_init, ev[0], ev[1]);
        cudaEventElapsedTime(&stats->ms_chains, ev[1], ev[2]);
        cudaEventElapsedTime(&stats->ms_finish, ev[2], ev[3]);
        stats->kernel_launches = c.launches;
    }
    cleanup();
    return ok ? KVP_OK : KVP_ERR_INTERNAL;
}

extern "C" int kvp_anneal_chain_state(kvp_problem* p, const kvp_anneal_params* a, uint32_t chain, uint64_t upto_moves,
                                      uint32_t* schedule, kvp_chain_result* result, void* stream)
{
    if (!schedule) return KVP_ERR_ARG;
    Ctx c;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc = prepare(p, a, st, c);
    if (rc) return rc;
    if (upto_moves > a->moves) upto_moves = a->moves;
    kvp_chain_result* res_dev = c.results;
    if (upto_moves == 0) {
        kvp_chain_result r0;
        memset(&r0, 0, sizeof r0);
        r0.best_ticks = r0.final_ticks = c.init_ticks; r0.best_move = ~0ull;
        KVP_CUDA(cudaMemcpyAsync(res_dev, &r0, sizeof r0, cudaMemcpyHostToDevice, st));
    }
    if ((rc = replay_to_sched(p, c, chain, upto_moves, res_dev))) return rc;
    KVP_CUDA(cudaMemcpyAsync(schedule, c.sched, (size_t)p->S * p->W32 * 4, cudaMemcpyDeviceToDevice, st));
    if (result) KVP_CUDA(cudaMemcpyAsync(result, res_dev, sizeof *result, cudaMemcpyDeviceToHost, st));
    KVP_CUDA(cudaStreamSynchronize(st));
    return KVP_OK;
}
