// Policy kernels: the look-ahead placement policy of Section III-B (window W, migration ratio R) evaluated for
// many (W, R) pairs at once, and the paper's own annealer that walks the (W, R) grid.
//
// A policy is sequential in the steps, so one CTA simulates one (W, R) pair from the first step to the last; the
// grid of pairs is the parallel axis. Per step the CTA (1) counts, for every unit, its accesses in the next W steps
// straight from the time-packed access columns (a 64-bit window and two popc), (2) histograms those frequencies
// separately for resident and non-resident units, (3) lets one thread walk the two histograms to find how many
// candidates fill free capacity, how many candidate/resident pairs are swapped and the frequency thresholds of
// both sets, (4) ranks the ties at the two thresholds by unit index with ballots, and (5) writes the new row.
#include <math.h>
#include <string.h>

#include <vector>

#include "kvp_common.cuh"

namespace kvp {

namespace {

constexpr uint32_t kMaxWindow = 64;
constexpr uint32_t kPolicyMaxUnits = 32768;
constexpr uint32_t TAG_WR = 5;

struct PolicyCtl {               // written by thread 0 once per step
    uint32_t fcs, takeC;         // candidates enter when f > fcs, or f == fcs and index rank < takeC
    uint32_t frs, takeR;         // residents leave when f < frs, or f == frs and index rank < takeR
};

// accesses of a unit in steps s .. s+W-1 (bits beyond the horizon are 0 in storage)
__device__ __forceinline__ uint32_t window_freq(const uint32_t* __restrict__ col, uint32_t S32, uint32_t s, uint32_t W)
{
    const uint32_t i0 = s >> 5, sh = s & 31u;
    const uint32_t w0 = __ldg(col + i0);
    const uint32_t w1 = i0 + 1 < S32 ? __ldg(col + i0 + 1) : 0u;
    const uint32_t w2 = i0 + 2 < S32 ? __ldg(col + i0 + 2) : 0u;
    uint32_t lo = __funnelshift_r(w0, w1, sh), hi = __funnelshift_r(w1, w2, sh);
    if (W < 32) { lo &= (1u << W) - 1u; hi = 0; }
    else if (W < 64) hi &= (1u << (W - 32)) - 1u;
    return __popc(lo) + __popc(hi);
}

// The kernel also serves Page Granularity Scheduling: then an "entity" is a page of `page` consecutive units (a power
// of two <= 32), its frequency is the number of its units the current step reads (W = 1), R = 1, the capacity is in
// pages, the initial placement is the first pages, and each row is expanded from the page bitmap.
// E entities, EW32 = ceil(E/32); for page == 1 entities are units and EW32 == W32.
__global__ void __launch_bounds__(1024)
lookahead_kernel(const uint32_t* __restrict__ Acol, const uint32_t* __restrict__ Arows, const uint32_t* __restrict__ row0,
                 uint32_t E, uint32_t page, uint32_t S, uint32_t S32, uint32_t W32, uint32_t EW32, uint32_t cap,
                 const uint32_t* __restrict__ windows, const uint32_t* __restrict__ ratios, uint32_t* __restrict__ out)
{
    extern __shared__ uint32_t sm[];
    uint32_t* H = sm;                                    // [EW32] resident bitmap over entities
    uint32_t* histC = H + EW32;                           // [66] candidates by frequency
    uint32_t* histR = histC + 66;                        // [66] residents by frequency
    uint32_t* warpC = histR + 66;                        // [32]
    uint32_t* warpR = warpC + 32;                        // [32]
    uint32_t* run = warpR + 32;                          // [2] ties already passed, candidates / residents
    PolicyCtl* ctl = reinterpret_cast<PolicyCtl*>(run + 2);
    uint8_t* fb = reinterpret_cast<uint8_t*>(ctl + 1);   // [rounds * T] frequency of every unit at this step

    const uint32_t T = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = T >> 5;
    const uint32_t W = page > 1 ? page : windows[blockIdx.x];          // W doubles as the largest frequency class
    const uint32_t permille = page > 1 ? 1000u : ratios[blockIdx.x];
    const uint32_t U = E;                                              // entities are indexed like units below
    const uint32_t rounds = (EW32 * 32 + T - 1) / T;
    uint32_t* mine = out + (size_t)blockIdx.x * S * W32;
    for (uint32_t i = tid; i < EW32; i += T) {
        if (row0) H[i] = __ldg(row0 + i);
        else H[i] = cap >= i * 32 + 32 ? 0xFFFFFFFFu : (cap > i * 32 ? (1u << (cap - i * 32)) - 1u : 0u);
    }
    __syncthreads();
    for (uint32_t s = 0; s < S; ++s) {
        for (uint32_t i = tid; i < 132; i += T) histC[i] = 0;          // both histograms
        if (tid == 0) { run[0] = 0; run[1] = 0; }
        __syncthreads();
        // frequencies and the two histograms (one shared-memory atomic per distinct class and warp)
        for (uint32_t j = 0; j < rounds; ++j) {
            const uint32_t u = j * T + tid;
            uint32_t f = 0, in = 0;
            if (u < U) {
                if (page > 1) {
                    const uint32_t first = u * page;                   // the page's units share one row word
                    const uint32_t word = __ldg(Arows + (size_t)s * W32 + (first >> 5)) >> (first & 31);
                    f = __popc(page == 32 ? word : word & ((1u << page) - 1u));
                } else {
                    f = window_freq(Acol + (size_t)u * S32, S32, s, W);
                }
                in = (H[u >> 5] >> (u & 31)) & 1u;
            }
            fb[u] = (uint8_t)f;
            const uint32_t key = u < U ? (f | (in << 7)) : 0xFFFFu;
            const uint32_t peers = __match_any_sync(0xFFFFFFFFu, key);
            if (u < U && lane == (uint32_t)(__ffs(peers) - 1)) {
                if (in) atomicAdd(histR + f, __popc(peers));
                else if (f) atomicAdd(histC + f, __popc(peers));
            }
        }
        __syncthreads();
        if (tid == 0) {
            uint32_t nC = 0, nR = 0;
            for (uint32_t f = 1; f <= W; ++f) nC += histC[f];
            for (uint32_t f = 0; f <= W; ++f) nR += histR[f];
            const uint32_t k = (uint32_t)(((uint64_t)nC * permille) / 1000u);
            const uint32_t free_slots = cap - nR;
            const uint32_t insf = min(k, free_slots), kb = k - insf;
            uint32_t cf = W, cl = histC[W], skip = insf;
            while (skip > 0) {                           // the best candidates take the free capacity
                if (cl == 0) { --cf; cl = histC[cf]; continue; }
                const uint32_t t = min(skip, cl);
                cl -= t; skip -= t;
            }
            uint32_t vf = 0, vl = histR[0], swaps = 0;
            while (swaps < kb) {                         // then the next best replace the least wanted residents
                while (cl == 0 && cf > 1) { --cf; cl = histC[cf]; }
                if (cl == 0) break;
                while (vl == 0 && vf < W) { ++vf; vl = histR[vf]; }
                if (vl == 0 || !(vf < cf)) break;
                const uint32_t t = min(min(cl, vl), kb - swaps);
                swaps += t; cl -= t; vl -= t;
            }
            PolicyCtl c;
            c.fcs = W + 1; c.takeC = 0; c.frs = 0; c.takeR = 0;
            const uint32_t I = insf + swaps;
            if (I) {
                uint32_t acc = 0;
                for (uint32_t f = W; f >= 1; --f) {
                    if (acc + histC[f] >= I) { c.fcs = f; c.takeC = I - acc; break; }
                    acc += histC[f];
                }
            }
            if (swaps) {
                uint32_t acc = 0;
                for (uint32_t f = 0; f <= W; ++f) {
                    if (acc + histR[f] >= swaps) { c.frs = f; c.takeR = swaps - acc; break; }
                    acc += histR[f];
                }
            }
            *ctl = c;
        }
        __syncthreads();
        const PolicyCtl c = *ctl;
        // units of round j are consecutive over the CTA, so index order = (round, thread) order
        for (uint32_t j = 0; j < rounds; ++j) {
            const uint32_t u = j * T + tid;
            const bool ok = u < U;
            const uint32_t f = ok ? fb[u] : 0u;
            const bool in = ok && ((H[u >> 5] >> (u & 31)) & 1u);
            const bool tieC = ok && !in && f == c.fcs, tieR = in && f == c.frs;
            const uint32_t bc = __ballot_sync(0xFFFFFFFFu, tieC), br = __ballot_sync(0xFFFFFFFFu, tieR);
            if (lane == 0) { warpC[warp] = __popc(bc); warpR[warp] = __popc(br); }
            __syncthreads();
            uint32_t rankC = run[0], rankR = run[1];
            for (uint32_t w = 0; w < warp; ++w) { rankC += warpC[w]; rankR += warpR[w]; }
            rankC += __popc(bc & ((1u << lane) - 1u));
            rankR += __popc(br & ((1u << lane) - 1u));
            const bool enter = ok && !in && f >= 1 && (f > c.fcs || (tieC && rankC < c.takeC));
            const bool leave = in && (f < c.frs || (tieR && rankR < c.takeR));
            const uint32_t bits = __ballot_sync(0xFFFFFFFFu, (in && !leave) || enter);
            __syncthreads();                             // every thread has read H and the warp counts of this round
            if (lane == 0 && (u >> 5) < EW32) {
                H[u >> 5] = bits;
                if (page == 1) mine[(size_t)s * W32 + (u >> 5)] = bits;
            }
            if (tid == 0) {
                uint32_t a = 0, b = 0;
                for (uint32_t w = 0; w < nwarps; ++w) { a += warpC[w]; b += warpR[w]; }
                run[0] += a; run[1] += b;
            }
            __syncthreads();
        }
        if (page > 1) {                                  // every resident page contributes `page` ones to the row
            const uint32_t per_word = 32 / page;
            for (uint32_t w = tid; w < W32; w += T) {
                const uint32_t e0 = w * per_word;
                uint32_t eb = H[e0 >> 5] >> (e0 & 31), word = 0;
                const uint32_t ones = page == 32 ? 0xFFFFFFFFu : (1u << page) - 1u;
                for (uint32_t i = 0; i < per_word; ++i)
                    if ((eb >> i) & 1u) word |= ones << (i * page);
                mine[(size_t)s * W32 + w] = word;
            }
        }
    }
}

// Sum of a per-thread value over the CTA; every thread gets the result. Needs a zeroed shared counter per call.
__device__ __forceinline__ uint32_t cta_sum(uint32_t v, uint32_t* slot)
{
    v = __reduce_add_sync(0xFFFFFFFFu, v);
    if ((threadIdx.x & 31) == 0 && v) atomicAdd(slot, v);
    __syncthreads();
    return *slot;
}

// Reactive Scheduling (Section IV-A): promote on miss, evict the least recently used. One CTA walks the steps; row
// s+1 follows from row s and the accesses of step s. Per step: hits refresh their stamp; the first min(misses, cap)
// missed units in index order are promoted; they take free capacity first and then the places of the residents with
// the smallest (stamp, index), found by a bitwise search for the stamp threshold and a ballot ranking of the ties.
__global__ void __launch_bounds__(1024)
reactive_kernel(const uint32_t* __restrict__ Arows, const uint32_t* __restrict__ row0, uint32_t U, uint32_t S,
                uint32_t W32, uint32_t cap, uint32_t* __restrict__ out)
{
    extern __shared__ uint32_t sm[];
    uint32_t* H = sm;                                    // [W32]
    uint32_t* cnt = H + W32;                             // [24] block counters of one step
    uint32_t* warpV = cnt + 24;                          // [32]
    uint32_t* warpM = warpV + 32;                        // [32]
    uint32_t* run = warpM + 32;                          // [2]
    uint16_t* stamp = reinterpret_cast<uint16_t*>(run + 2);   // [rounds * T] step of last use + 1, 0 = never
    const uint32_t T = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = T >> 5;
    const uint32_t rounds = (W32 * 32 + T - 1) / T;
    for (uint32_t i = tid; i < W32; i += T) { H[i] = __ldg(row0 + i); out[i] = H[i]; }
    for (uint32_t i = tid; i < rounds * T; i += T) stamp[i] = 0;
    __syncthreads();
    for (uint32_t s = 0; s + 1 < S; ++s) {
        for (uint32_t i = tid; i < 24; i += T) cnt[i] = 0;
        if (tid == 0) { run[0] = 0; run[1] = 0; }
        __syncthreads();
        uint32_t my_miss = 0, my_res = 0;
        for (uint32_t j = 0; j < rounds; ++j) {
            const uint32_t u = j * T + tid;
            if (u < U) {
                const uint32_t a = (__ldg(Arows + (size_t)s * W32 + (u >> 5)) >> (u & 31)) & 1u;
                const uint32_t in = (H[u >> 5] >> (u & 31)) & 1u;
                if (a & in) stamp[u] = (uint16_t)(s + 1);
                my_miss += a & ~in & 1u;
                my_res += in;
            }
        }
        const uint32_t nM = cta_sum(my_miss, cnt + 0), nR = cta_sum(my_res, cnt + 1);
        const uint32_t promoted = min(nM, cap), free_slots = cap - nR;
        const uint32_t evict = promoted > free_slots ? promoted - free_slots : 0u;
        // smallest stamp value tau with |{resident, stamp <= tau}| >= evict, bit by bit from the top (stamps < 2^16)
        uint32_t tau = 0, takeV = 0;
        if (evict) {
            for (int bit = 15; bit >= 0; --bit) {
                const uint32_t probe = tau | (1u << bit);             // is the answer >= probe?  <=> count(stamp < probe) < evict
                uint32_t c = 0;
                for (uint32_t j = 0; j < rounds; ++j) {
                    const uint32_t u = j * T + tid;
                    if (u < U && ((H[u >> 5] >> (u & 31)) & 1u) && stamp[u] < probe) ++c;
                }
                if (cta_sum(c, cnt + 2 + (15 - bit)) < evict) tau = probe;
            }
            uint32_t c = 0;
            for (uint32_t j = 0; j < rounds; ++j) {
                const uint32_t u = j * T + tid;
                if (u < U && ((H[u >> 5] >> (u & 31)) & 1u) && stamp[u] < tau) ++c;
            }
            takeV = evict - cta_sum(c, cnt + 18);
        }
        __syncthreads();
        for (uint32_t j = 0; j < rounds; ++j) {
            const uint32_t u = j * T + tid;
            const bool ok = u < U;
            const bool in = ok && ((H[u >> 5] >> (u & 31)) & 1u);
            const bool a = ok && ((__ldg(Arows + (size_t)s * W32 + (u >> 5)) >> (u & 31)) & 1u);
            const uint32_t st = ok ? stamp[u] : 0u;
            const bool miss = a && !in, tieV = in && evict && st == tau;
            const uint32_t bv = __ballot_sync(0xFFFFFFFFu, tieV), bm = __ballot_sync(0xFFFFFFFFu, miss);
            if (lane == 0) { warpV[warp] = __popc(bv); warpM[warp] = __popc(bm); }
            __syncthreads();
            uint32_t rankV = run[0], rankM = run[1];
            for (uint32_t w = 0; w < warp; ++w) { rankV += warpV[w]; rankM += warpM[w]; }
            rankV += __popc(bv & ((1u << lane) - 1u));
            rankM += __popc(bm & ((1u << lane) - 1u));
            const bool leave = in && evict && (st < tau || (tieV && rankV < takeV));
            const bool enter = miss && rankM < promoted;
            if (enter) stamp[u] = (uint16_t)(s + 1);
            const uint32_t bits = __ballot_sync(0xFFFFFFFFu, (in && !leave) || enter);
            __syncthreads();
            if (lane == 0 && (u >> 5) < W32) { H[u >> 5] = bits; out[(size_t)(s + 1) * W32 + (u >> 5)] = bits; }
            if (tid == 0) {
                uint32_t x = 0, y = 0;
                for (uint32_t w = 0; w < nwarps; ++w) { x += warpV[w]; y += warpM[w]; }
                run[0] += x; run[1] += y;
            }
            __syncthreads();
        }
    }
}

struct WRK {
    const uint64_t* table; const uint32_t* acc; const uint32_t* shifts;
    uint32_t w_max, n_ratio, chains, levels, early_permille, w0, r0, seed_lo, seed_hi;
    uint64_t iters, per_level;
};

// The paper's annealer over (W, R): one thread per independent chain, the objective is a table lookup.
__global__ void wr_anneal_kernel(const WRK k, kvp_wr_result* __restrict__ results)
{
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= k.chains) return;
    const int dws[4] = {-2, -1, 1, 2};
    uint32_t w = k.w0, r = k.r0;
    uint64_t cur = k.table[(size_t)(w - 1) * k.n_ratio + r];
    kvp_wr_result res;
    res.best_ticks = cur; res.best_w = w; res.best_r = r; res.n_accepted = 0;
    uint64_t bab = cur, i = 0;
    uint32_t level = 0;
    uint64_t next_boundary = k.levels > 1 ? k.per_level : ~0ull;
    for (; i < k.iters; ++i) {
        if (i == next_boundary) {
            ++level;
            if (k.early_permille && (bab - res.best_ticks) * 1000ull < bab * (uint64_t)k.early_permille) break;
            bab = res.best_ticks;
            next_boundary = level + 1 < k.levels ? next_boundary + k.per_level : ~0ull;
        }
        uint32_t x[4];
        philox4x32_10((uint32_t)i, (uint32_t)(i >> 32), c, TAG_WR, k.seed_lo, k.seed_hi, x);
        const uint32_t sel = x[0] & 255u;
        const int op = sel < 102u ? 0 : (sel < 204u ? 1 : 2);            // window, ratio, diagonal: 0.4, 0.4, 0.2
        const int dw = op != 1 ? dws[(x[0] >> 8) & 3u] : 0;
        const int dr = op != 0 ? (((x[0] >> 10) & 1u) ? 1 : -1) : 0;
        const int nw = (int)w + dw, nr = (int)r + dr;
        if (nw < 1 || nw > (int)k.w_max || nr < 0 || nr >= (int)k.n_ratio) continue;   // off the grid: discarded
        const uint64_t cand = k.table[(size_t)(nw - 1) * k.n_ratio + nr];
        bool accept = cand <= cur;
        if (!accept) {
            const uint64_t q = (cand - cur) >> k.shifts[level];
            accept = q < KVP_TABLE_Q && x[3] < k.acc[(size_t)level * KVP_TABLE_Q + q];  // Metropolis
        }
        if (!accept) continue;
        ++res.n_accepted;
        w = (uint32_t)nw; r = (uint32_t)nr; cur = cand;
        if (cur < res.best_ticks) { res.best_ticks = cur; res.best_w = w; res.best_r = r; }
    }
    res.iters_done = i; res.final_ticks = cur; res.final_w = w; res.final_r = r;
    results[c] = res;
}

}  // namespace

}  // namespace kvp

using namespace kvp;

static size_t policy_smem(uint32_t EW32, uint32_t rounds, uint32_t T)
{
    return ((size_t)EW32 + 66 + 66 + 32 + 32 + 2 + 4) * 4 + (size_t)rounds * T;
}

extern "C" int kvp_policy_reactive(kvp_problem* p, uint32_t init_mode, uint32_t* schedule, void* stream)
{
    if (!p || !schedule || init_mode > KVP_INIT_STATIC_FREQ || p->dL) return KVP_ERR_ARG;   // fixed populations only
    if (p->U > kPolicyMaxUnits) return KVP_ERR_RANGE;        // stamps are 16 bits and live in shared memory
    KVP_CUDA(cudaSetDevice(p->device));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    uint32_t T = (p->U + 31) / 32 * 32;
    if (T > 1024) T = 1024;
    const uint32_t rounds = (p->W32 * 32 + T - 1) / T;
    const size_t smem = ((size_t)p->W32 + 24 + 32 + 32 + 2) * 4 + (size_t)rounds * T * 2;
    const uint32_t* row = p->d_row_freq;
    if (init_mode == KVP_INIT_STATIC_FIRST) {
        int rc = ensure_scratch(p, (size_t)p->W32 * 4, st);
        if (rc) return rc;
        if ((rc = launch_static_first_row(p, static_cast<uint32_t*>(p->d_scratch), st))) return rc;
        row = static_cast<uint32_t*>(p->d_scratch);
    }
    KVP_CUDA(cudaFuncSetAttribute(reactive_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    reactive_kernel<<<1, T, smem, st>>>(p->dA, row, p->U, p->S, p->W32, p->cap, schedule);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

extern "C" int kvp_policy_page(kvp_problem* p, uint32_t page_units, uint32_t* schedule, void* stream)
{
    if (p && p->dL) return KVP_ERR_ARG;                      // fixed populations only
    if (!p || !schedule || page_units < 2 || page_units > 32 || (page_units & (page_units - 1)) || p->U % page_units)
        return KVP_ERR_ARG;
    if (p->U > kPolicyMaxUnits) return KVP_ERR_RANGE;
    KVP_CUDA(cudaSetDevice(p->device));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    const uint32_t E = p->U / page_units, EW32 = (E + 31) / 32;
    uint32_t T = (E + 31) / 32 * 32;
    if (T > 1024) T = 1024;
    const uint32_t rounds = (EW32 * 32 + T - 1) / T;
    const size_t smem = policy_smem(EW32, rounds, T);
    KVP_CUDA(cudaFuncSetAttribute(lookahead_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    lookahead_kernel<<<1, T, smem, st>>>(p->dAcol, p->dA, nullptr, E, page_units, p->S, p->S32, p->W32, EW32,
                                         p->cap / page_units, nullptr, nullptr, schedule);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

extern "C" int kvp_policy_lookahead(kvp_problem* p, uint32_t init_mode, const uint32_t* windows, const uint32_t* ratios_permille,
                                    uint32_t n, uint32_t* schedules, void* stream)
{
    if (!p || !windows || !ratios_permille || !schedules || !n || init_mode > KVP_INIT_STATIC_FREQ) return KVP_ERR_ARG;
    if (p->dL) return KVP_ERR_ARG;                           // fixed populations only
    for (uint32_t i = 0; i < n; ++i)
        if (windows[i] < 1 || windows[i] > kMaxWindow || ratios_permille[i] > 1000) return KVP_ERR_ARG;
    if (p->U > kPolicyMaxUnits) return KVP_ERR_RANGE;
    KVP_CUDA(cudaSetDevice(p->device));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    uint32_t T = (p->U + 31) / 32 * 32;
    if (T > 1024) T = 1024;
    const uint32_t rounds = (p->W32 * 32 + T - 1) / T;
    const size_t smem = policy_smem(p->W32, rounds, T);
    // per-call parameters and, for the first-come placement, its row
    int rc = ensure_scratch(p, ((size_t)2 * n + p->W32) * 4 + 256, st);
    if (rc) return rc;
    uint32_t* d_w = static_cast<uint32_t*>(p->d_scratch);
    uint32_t* d_r = d_w + n;
    uint32_t* d_row = d_r + n + ((64 - (2 * n) % 64) % 64);          // keep the row 256-byte aligned
    KVP_CUDA(cudaMemcpyAsync(d_w, windows, (size_t)n * 4, cudaMemcpyHostToDevice, st));
    KVP_CUDA(cudaMemcpyAsync(d_r, ratios_permille, (size_t)n * 4, cudaMemcpyHostToDevice, st));
    const uint32_t* row = p->d_row_freq;
    if (init_mode == KVP_INIT_STATIC_FIRST) {
        if ((rc = launch_static_first_row(p, d_row, st))) return rc;
        row = d_row;
    }
    KVP_CUDA(cudaFuncSetAttribute(lookahead_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    lookahead_kernel<<<n, T, smem, st>>>(p->dAcol, p->dA, row, p->U, 1u, p->S, p->S32, p->W32, p->W32, p->cap, d_w, d_r,
                                         schedules);
    KVP_CUDA(cudaGetLastError());
    KVP_CUDA(cudaStreamSynchronize(st));                             // the host arrays may go away
    return KVP_OK;
}

extern "C" int kvp_wr_grid(kvp_problem* p, uint32_t init_mode, uint32_t w_max, uint32_t n_ratio, uint64_t* table, void* stream)
{
    if (!p || !table || w_max < 1 || w_max > kMaxWindow || n_ratio < 2 || n_ratio > 1001 || p->dL) return KVP_ERR_ARG;
    if (p->U > kPolicyMaxUnits) return KVP_ERR_RANGE;
    KVP_CUDA(cudaSetDevice(p->device));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    const uint32_t total = w_max * n_ratio;
    const size_t sched_bytes = (size_t)p->S * p->W32 * 4;
    uint32_t chunk = (uint32_t)(((size_t)1 << 30) / sched_bytes);    // at most 1 GiB of schedules at a time
    if (chunk < 1) chunk = 1;
    if (chunk > total) chunk = total;
    uint32_t* scheds = nullptr;
    KVP_CUDA(cudaMallocAsync(&scheds, (size_t)chunk * sched_bytes, st));
    std::vector<uint32_t> ws(total), rs(total);
    for (uint32_t i = 0; i < total; ++i) { ws[i] = i / n_ratio + 1; rs[i] = (1000u * (i % n_ratio)) / (n_ratio - 1); }
    int rc = KVP_OK;
    for (uint32_t i = 0; i < total && !rc; i += chunk) {
        const uint32_t m = total - i < chunk ? total - i : chunk;
        rc = kvp_policy_lookahead(p, init_mode, ws.data() + i, rs.data() + i, m, scheds, stream);
        if (!rc) rc = kvp_eval(p, scheds, m, nullptr, table + i, nullptr, nullptr, nullptr, stream);
    }
    cudaFreeAsync(scheds, st);
    return rc;
}

extern "C" int kvp_wr_anneal(const uint64_t* table, uint32_t w_max, uint32_t n_ratio, const kvp_wr_params* wp,
                             kvp_wr_result* results, kvp_wr_result* best, void* stream)
{
    if (!table || !wp || w_max < 1 || n_ratio < 2) return KVP_ERR_ARG;
    if (!wp->chains || !wp->levels || wp->levels > 4096 || !wp->iters || wp->reserved) return KVP_ERR_ARG;
    if (wp->w0 < 1 || wp->w0 > w_max || wp->r0 >= n_ratio) return KVP_ERR_ARG;
    if (!(wp->p0 > 0.0 && wp->p0 < 1.0) || !(wp->alpha > 0.0 && wp->alpha <= 1.0)) return KVP_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // temperature ladder from the table itself: the mean uphill step between grid neighbours is accepted with p0
    const size_t cells = (size_t)w_max * n_ratio;
    std::vector<uint64_t> T(cells);
    KVP_CUDA(cudaMemcpyAsync(T.data(), table, cells * 8, cudaMemcpyDeviceToHost, st));
    KVP_CUDA(cudaStreamSynchronize(st));
    const int dws[4] = {-2, -1, 1, 2};
    uint64_t sum = 0, cnt = 0;
    for (uint32_t w = 1; w <= w_max; ++w)
        for (uint32_t r = 0; r < n_ratio; ++r)
            for (int op = 0; op < 3; ++op)
                for (int a = 0; a < 4; ++a)
                    for (int b = 0; b < 2; ++b) {
                        if ((op == 0 && b) || (op == 1 && a)) continue;
                        const long nw = (long)w + (op != 1 ? dws[a] : 0), nr = (long)r + (op != 0 ? (b ? 1 : -1) : 0);
                        if (nw < 1 || nw > (long)w_max || nr < 0 || nr >= (long)n_ratio) continue;
                        const uint64_t t0 = T[(size_t)(w - 1) * n_ratio + r], t1 = T[(size_t)(nw - 1) * n_ratio + nr];
                        if (t1 > t0) { sum += t1 - t0; ++cnt; }
                    }
    uint64_t mean = cnt ? sum / cnt : 1;
    if (!mean) mean = 1;
    std::vector<double> temps(wp->levels);
    double C = -(double)mean / log(wp->p0);
    for (uint32_t j = 0; j < wp->levels; ++j) { temps[j] = C; C = C * wp->alpha; }
    std::vector<uint32_t> acc((size_t)wp->levels * KVP_TABLE_Q), shifts(wp->levels);
    int rc = kvp_accept_table(temps.data(), wp->levels, acc.data(), shifts.data());
    if (rc) return rc;
    char* dev = nullptr;
    const size_t acc_bytes = acc.size() * 4, sh_bytes = (shifts.size() * 4 + 255) & ~(size_t)255;
    const size_t res_bytes = (size_t)wp->chains * sizeof(kvp_wr_result);
    KVP_CUDA(cudaMallocAsync(&dev, acc_bytes + sh_bytes + res_bytes, st));
    cudaError_t ce = cudaMemcpyAsync(dev, acc.data(), acc_bytes, cudaMemcpyHostToDevice, st);
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(dev + acc_bytes, shifts.data(), shifts.size() * 4, cudaMemcpyHostToDevice, st);
    if (ce != cudaSuccess) {
        cudaFreeAsync(dev, st);
        KVP_CUDA(ce);
    }
    WRK k;
    k.table = table; k.acc = (const uint32_t*)dev; k.shifts = (const uint32_t*)(dev + acc_bytes);
    k.w_max = w_max; k.n_ratio = n_ratio; k.chains = wp->chains; k.levels = wp->levels;
    k.early_permille = wp->early_stop_permille; k.w0 = wp->w0; k.r0 = wp->r0;
    k.seed_lo = (uint32_t)wp->seed; k.seed_hi = (uint32_t)(wp->seed >> 32);
    k.iters = wp->iters; k.per_level = wp->iters / wp->levels ? wp->iters / wp->levels : 1;
    kvp_wr_result* d_res = (kvp_wr_result*)(dev + acc_bytes + sh_bytes);
    wr_anneal_kernel<<<(wp->chains + 127) / 128, 128, 0, st>>>(k, d_res);
    cudaError_t le = cudaGetLastError();
    std::vector<kvp_wr_result> host(wp->chains);
    if (le == cudaSuccess) le = cudaMemcpyAsync(host.data(), d_res, res_bytes, cudaMemcpyDeviceToHost, st);
    cudaFreeAsync(dev, st);
    KVP_CUDA(le);
    KVP_CUDA(cudaStreamSynchronize(st));
    if (results) memcpy(results, host.data(), res_bytes);
    if (best) {
        *best = host[0];
        for (uint32_t c = 1; c < wp->chains; ++c)
            if (host[c].best_ticks < best->best_ticks) *best = host[c];
    }
    return KVP_OK;
}
