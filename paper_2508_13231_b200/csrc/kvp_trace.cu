// Trace kernels: synthetic importance per unit and step, top-k per (layer, kv-head) group, packed into uint32
// bitmaps. Two passes by default: the first writes a score matrix (large traces: a thread per unit walks the steps;
// small ones: the draws in parallel over units and steps, the AR(1) recurrence, sequential in time, by one lane per
// unit); then one CTA per (group, step) finds the k-th largest score: the first eight bits of its range by a
// shared-memory histogram, the rest by ranking the keys of that bin, ties going to the lower unit index. A fused single-pass form
// (one CTA per group walking the steps, state in registers) serves layered or growing traces and those whose score
// matrix would exceed the scratch budget.
#include "kvp_common.cuh"

namespace kvp {

namespace {

struct TraceK {
    uint32_t groups, n, steps, topk, W32;
    PhiloxKeys keys;         // round keys of the seed
    int32_t rho_q, c_q, sigma_q, burst_jump;
    uint32_t burst_thr;
    const int32_t* base;
    uint32_t* out;
    int aligned;             // n % 32 == 0: whole output words belong to one group
    uint32_t layers;         // >= 1; step t belongs to token t / layers and layer t % layers
    uint32_t per_layer;      // groups per layer
    const uint32_t* birth;   // or null: unit u can be read from step birth[u] on
};

// Irwin-Hall(8) noise with unit variance in Q16.16: the sum of the eight 16-bit halves of one Philox block, centred
// and scaled by floor(). |result| <= 321,057, so 32 bits hold it; only the product needs 64.
__device__ __forceinline__ int32_t noise_q16(const PhiloxKeys& keys, uint32_t u, uint32_t t)
{
    uint32_t r[4];
    philox4x32_10(u, t, 0u, TAG_NOISE, keys, r);
    uint32_t sum = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) sum = __dp2a_lo(r[i], 0x0101u, sum);      // + low half + high half
    const int64_t scaled = (int64_t)((int32_t)sum - 262140) * 80265;
    return (int32_t)(scaled >> 16);                                       // arithmetic shift = floor
}

// Sum of a per-thread value over the CTA; every thread gets the result. slot: one of 32 shared counters.
__device__ __forceinline__ uint32_t block_sum(uint32_t v, uint32_t* slot)
{
    v = __reduce_add_sync(0xFFFFFFFFu, v);
    if ((threadIdx.x & 31) == 0 && v) atomicAdd(slot, v);
    __syncthreads();
    return *slot;
}

constexpr int kDigitBits = 8;                        // the search fixes this many bits of the threshold per pass
constexpr int kBins = 1 << kDigitBits;
constexpr int kPasses = 32 / kDigitBits;
constexpr uint32_t kListCap = 256;                   // a threshold bin of up to this many keys is finished by ranking

struct SelectSmem {
    uint32_t hist[kPasses][kBins];   // per pass: how many keys with the threshold's higher bits have each digit
    uint32_t cnt[4];                 // block-wide counts beside the search ([1]: keys in `list`)
    uint32_t list[kListCap];         // the keys of the threshold's bin after the first pass
    uint32_t warp[32];
    uint32_t run;
    uint32_t hi, lo;                 // largest and smallest key of the step
    uint32_t K, need, equal;         // threshold so far, how many keys are still to find at or below it, ties at it
};

// State of one selection; a barrier must follow before select_step.
__device__ __forceinline__ void select_reset(SelectSmem& sm)
{
    for (uint32_t i = threadIdx.x; i < kPasses * kBins; i += blockDim.x) (&sm.hist[0][0])[i] = 0;
    if (threadIdx.x < 4) sm.cnt[threadIdx.x] = 0;
    if (threadIdx.x == 0) { sm.hi = 0u; sm.lo = ~0u; }
}

// Top-k of one (group, step): the CTA holds the n keys (UPT per thread, unit i = j*T + tid, 0 past n) and sets the
// bits of the k largest, ties to the lower unit index. select_reset and a barrier come first.
// topk: how many to pick (at most the number of non-zero keys when zero marks a unit that is not there yet).
//
// The threshold K (the k-th largest key) is found digit by digit from the top, eight bits per pass: the keys that
// agree with K in the bits fixed so far are counted per digit in a shared-memory histogram, and one warp walks
// the histogram from the top until the counts reach what is still needed. The search works on the keys minus the
// smallest one, so only the bits of (largest - smallest) need a pass: three passes on these scores.
// FULL: the CTA's UPT * T slots are exactly the n units, so no slot needs a bounds test.
template <int UPT, bool FULL = false>
__device__ __forceinline__ void select_step(const uint32_t (&key)[UPT], const TraceK& k, uint32_t topk, uint32_t gbase,
                                            uint32_t t, SelectSmem& sm)
{
    const uint32_t T = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t mx = 0u, mn = ~0u;
#pragma unroll
    for (int j = 0; j < UPT; ++j)
        if (FULL || j * T + tid < k.n) { mx = max(mx, key[j]); mn = min(mn, key[j]); }
    mx = __reduce_max_sync(0xFFFFFFFFu, mx);
    mn = __reduce_min_sync(0xFFFFFFFFu, mn);
    if (lane == 0) { atomicMax(&sm.hi, mx); atomicMin(&sm.lo, mn); }
    __syncthreads();
    // The search runs on key - smallest key: the same order, and the digits then spread over the range the keys
    // really cover (scores on both sides of zero differ in every leading bit, although they span twenty bits or so:
    // as raw keys they would need four passes, the first two with nearly all keys in two or three bins).
    const uint32_t lo = sm.lo;
    uint32_t kk[UPT];
#pragma unroll
    for (int j = 0; j < UPT; ++j) kk[j] = key[j] - lo;
    int rem = 32 - __clz(sm.hi - lo);                        // bits still open; 0 when all keys are equal
    uint32_t K = 0u;                                         // the bits above them are zero in every reduced key
    uint32_t need = topk, equal = k.n;                       // all keys equal: every one ties at K
    for (int pass = 0; rem > 0; ++pass) {
        const int w = rem < kDigitBits ? rem : kDigitBits, sh = rem - w;
        uint32_t* hist = sm.hist[pass];
        if (pass == 0) {                                     // no reduced key has a bit above the open ones: all count
#pragma unroll
            for (int j = 0; j < UPT; ++j)
                if (FULL || j * T + tid < k.n) atomicAdd(hist + (kk[j] >> sh), 1u);
        } else {
#pragma unroll
            for (int j = 0; j < UPT; ++j) {
                const bool in = (FULL || j * T + tid < k.n) && (kk[j] >> rem) == (K >> rem);
                if (in) atomicAdd(hist + ((kk[j] >> sh) & ((1u << w) - 1u)), 1u);
            }
        }
        __syncthreads();
        if (warp == 0) {
            // lane l owns digits 8l .. 8l+7; suffix sums over the lanes, then over the owner's eight bins
            uint32_t h[8], s = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { h[i] = hist[8 * lane + i]; s += h[i]; }
            uint32_t suf = s;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t v = __shfl_down_sync(0xFFFFFFFFu, suf, off);
                if (lane + off < 32) suf += v;
            }
            const uint32_t reach = __ballot_sync(0xFFFFFFFFu, suf >= need);    // never empty: the counts add up to >= need
            if (lane == 31u - __clz(reach)) {
                uint32_t higher = suf - s;
#pragma unroll
                for (int i = 7; i >= 0; --i) {
                    if (higher + h[i] >= need) {
                        sm.K = K | ((uint32_t)(8 * lane + i) << sh);
                        sm.need = need - higher;
                        sm.equal = h[i];
                        break;
                    }
                    higher += h[i];
                }
            }
        }
        __syncthreads();
        K = sm.K; need = sm.need; equal = sm.equal;
        rem = sh;
        if (pass == 0 && rem > 0 && equal <= kListCap) {
            // The first digit's bin usually holds a few dozen keys: they go to a shared list and each is ranked against
            // the others, which settles the remaining bits at once; further histogram passes, in which every thread
            // tests all of its keys again, are left to bins with many keys (ties).
#pragma unroll
            for (int j = 0; j < UPT; ++j)
                if ((FULL || j * T + tid < k.n) && (kk[j] >> rem) == (K >> rem)) sm.list[atomicAdd(&sm.cnt[1], 1u)] = kk[j];
            __syncthreads();
            for (uint32_t c = tid; c < equal; c += T) {
                const uint32_t v = sm.list[c];
                uint32_t above = 0, same = 0;
                for (uint32_t i = 0; i < equal; ++i) {
                    const uint32_t x = sm.list[i];
                    above += x > v ? 1u : 0u;
                    same += x == v ? 1u : 0u;
                }
                if (above < need && need <= above + same) {   // v is the need-th largest; equal keys write the same
                    sm.K = v; sm.need = need - above; sm.equal = same;
                }
            }
            __syncthreads();
            K = sm.K; need = sm.need; equal = sm.equal;
            rem = 0;
        }
    }
    const uint32_t take = need;                              // ties to admit, lowest unit index first
    const bool rank_ties = equal != take;
    uint32_t* row = k.out + (size_t)t * k.W32;
    auto emit = [&](int j, bool pick) {
        const uint32_t i = j * T + tid;
        if (k.aligned) {
            const uint32_t bits = __ballot_sync(0xFFFFFFFFu, pick);
            if (lane == 0 && (FULL || j * T + (tid & ~31u) < k.n)) row[(gbase + j * T + tid) >> 5] = bits;
        } else if (pick) {
            atomicOr(row + ((gbase + i) >> 5), 1u << ((gbase + i) & 31));
        }
    };
    if (!rank_ties) {                                        // the usual case, kept apart so that its loop stays small
#pragma unroll
        for (int j = 0; j < UPT; ++j) emit(j, (FULL || j * T + tid < k.n) && kk[j] >= K);
        return;
    }
    if (tid == 0) sm.run = 0;
    __syncthreads();
#pragma unroll
    for (int j = 0; j < UPT; ++j) {
        const uint32_t i = j * T + tid;
        const bool ok = FULL || i < k.n;
        const bool tie = ok && kk[j] == K;
        // units of round j are consecutive over the CTA, so index order = (round, thread) order
        const uint32_t tb = __ballot_sync(0xFFFFFFFFu, tie);
        if (lane == 0) sm.warp[warp] = __popc(tb);
        __syncthreads();
        uint32_t before = sm.run;
        for (uint32_t w = 0; w < warp; ++w) before += sm.warp[w];
        before += __popc(tb & ((1u << lane) - 1u));
        const bool pick = (ok && kk[j] > K) || (tie && before < take);
        __syncthreads();
        if (tid == 0) { uint32_t s = 0; for (uint32_t w = 0; w < (T >> 5); ++w) s += sm.warp[w]; sm.run += s; }
        __syncthreads();
        emit(j, pick);
    }
}

// importance of unit u at step t given its state at t-1 (Q16.16). The 64-bit sum of the two 32x32 products is
// shifted and then cut to 32 bits (the range check on the host keeps the true value inside them).
__device__ __forceinline__ int32_t next_state(const TraceK& k, uint32_t u, uint32_t t, int32_t x)
{
    const int32_t e = noise_q16(k.keys, u, t);
    const int64_t acc = t == 0 ? (int64_t)k.sigma_q * e : (int64_t)k.rho_q * x + (int64_t)k.c_q * e;
    int32_t xn = (int32_t)(acc >> 16);
    if (k.burst_thr) {
        uint32_t r[4];
        philox4x32_10(u, t, 0u, TAG_BURST, k.keys, r);
        if (r[0] < k.burst_thr) xn += k.burst_jump;
    }
    return xn;
}

// Fused form: one CTA per group walks the steps; used when the score matrix would not fit the scratch budget.
// Two CTAs per SM (at most 32 registers per thread): one CTA's barriers in the search hide behind the other's work.
// GROW: units have birth steps; one that is not there yet gets key 0 and is never picked.
template <int UPT, bool GROW>
__global__ void __launch_bounds__(1024, 2)
trace_kernel(const TraceK k)
{
    __shared__ SelectSmem sm;
    const uint32_t g = blockIdx.x, T = blockDim.x, tid = threadIdx.x;
    const uint32_t gbase = g * k.n;
    int32_t x[UPT], b[UPT];
#pragma unroll
    for (int j = 0; j < UPT; ++j) {
        const uint32_t i = j * T + tid;
        x[j] = 0;
        b[j] = (i < k.n && k.base) ? __ldg(k.base + gbase + i) : 0;
    }
    // the group reads at the steps of its layer, one per token
    const uint32_t layer = g / k.per_layer;
    uint32_t born[GROW ? UPT : 1];
    if (GROW) {
#pragma unroll
        for (int j = 0; j < (GROW ? UPT : 1); ++j) {
            const uint32_t i = j * T + tid;
            born[j] = i < k.n ? __ldg(k.birth + gbase + i) : 0u;
        }
    }
    for (uint32_t tok = 0, t = layer; t < k.steps; ++tok, t += k.layers) {
        select_reset(sm);
        uint32_t key[UPT], here = 0;
#pragma unroll
        for (int j = 0; j < UPT; ++j) {
            const uint32_t i = j * T + tid;
            key[j] = 0;
            if (i < k.n) {
                x[j] = next_state(k, gbase + i, tok, x[j]);
                if (!GROW || born[GROW ? j : 0] <= t) {
                    key[j] = (uint32_t)(x[j] + b[j]) ^ 0x80000000u;   // order-preserving map int32 -> uint32, never 0
                    ++here;
                }
            }
        }
        __syncthreads();
        uint32_t topk = k.topk;
        if (GROW) topk = min(topk, block_sum(here, &sm.cnt[0]));
        select_step<UPT>(key, k, topk, gbase, t, sm);
        __syncthreads();
    }
}

// Two-pass form, pass 1: scores [steps][U]. The random draws of a (unit, step) pair depend on nothing else, only the
// AR(1) recurrence is sequential in time. A CTA owns 32 consecutive units and walks the steps in segments: all its
// threads draw the segment's noise (and burst decisions) into shared memory, then one warp, a lane per unit, runs
// the recurrence over the segment and writes 128 contiguous bytes per step. 256 threads: while the one warp runs
// the recurrence the others wait, so smaller CTAs waste less (640 x 4096 units x 64 steps: 0.95 ms with 512, 0.85 with 256).
constexpr uint32_t kScoreSeg = 256, kScoreThreads = 256;

__global__ void __launch_bounds__(kScoreThreads)
trace_scores_kernel(const TraceK k, uint32_t U, int32_t* __restrict__ scores)
{
    __shared__ int32_t draw[kScoreSeg][32];              // noise << 1 | burst
    const uint32_t u0 = blockIdx.x * 32, tid = threadIdx.x;
    const uint32_t ul = tid & 31, u = u0 + ul;
    int32_t x = 0, b = 0;
    if (tid < 32 && u < U && k.base) b = __ldg(k.base + u);
    for (uint32_t t0 = 0; t0 < k.steps; t0 += kScoreSeg) {
        const uint32_t len = min(kScoreSeg, k.steps - t0);
        for (uint32_t tt = tid >> 5; tt < len; tt += kScoreThreads / 32) {
            if (u < U) {
                int32_t d = noise_q16(k.keys, u, t0 + tt) * 2;
                if (k.burst_thr) {
                    uint32_t r[4];
                    philox4x32_10(u, t0 + tt, 0u, TAG_BURST, k.keys, r);
                    d |= r[0] < k.burst_thr ? 1 : 0;
                }
                draw[tt][ul] = d;
            }
        }
        __syncthreads();
        if (tid < 32 && u < U) {
            for (uint32_t tt = 0; tt < len; ++tt) {
                const int32_t d = draw[tt][ul], e = d >> 1;
                const uint32_t t = t0 + tt;
                const int64_t acc = t == 0 ? (int64_t)k.sigma_q * e : (int64_t)k.rho_q * x + (int64_t)k.c_q * e;
                x = (int32_t)(acc >> 16);
                if (d & 1) x += k.burst_jump;
                scores[(size_t)t * U + u] = x + b;
            }
        }
        __syncthreads();
    }
}

// Pass 1 for traces of many units: a thread per unit walks the steps, draws and recurrence together, and the threads
// of a warp write 128 contiguous bytes per step. No shared memory and no barrier; the draws of later steps do not
// depend on the state, so the loop, unrolled eight times (3% faster than four), overlaps their Philox chains with the
// recurrence. It needs about a
// thousand units per SM to fill the machine, which is why fewer units take the segmented kernel above.
__global__ void __launch_bounds__(256)
trace_scores_unit_kernel(const TraceK k, uint32_t U, int32_t* __restrict__ scores)
{
    const uint32_t u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= U) return;
    const int32_t b = k.base ? __ldg(k.base + u) : 0;
    int32_t x = 0;
#pragma unroll 8
    for (uint32_t t = 0; t < k.steps; ++t) {
        x = next_state(k, u, t, x);
        scores[(size_t)t * U + u] = x + b;
    }
}

// Two-pass form, pass 2: the top-k selections of different steps are independent: one CTA per (group, step).
template <int UPT, bool FULL>
__global__ void __launch_bounds__(1024)
trace_select_kernel(const TraceK k, uint32_t U, const int32_t* __restrict__ scores)
{
    __shared__ SelectSmem sm;
    const uint32_t g = blockIdx.x, t = blockIdx.y, T = blockDim.x, tid = threadIdx.x;
    const uint32_t gbase = g * k.n;
    select_reset(sm);
    uint32_t key[UPT];
#pragma unroll
    for (int j = 0; j < UPT; ++j) {
        const uint32_t i = j * T + tid;
        key[j] = (FULL || i < k.n) ? (uint32_t)__ldg(scores + (size_t)t * U + gbase + i) ^ 0x80000000u : 0u;
    }
    __syncthreads();
    select_step<UPT, FULL>(key, k, k.topk, gbase, t, sm);
}

}  // namespace

}  // namespace kvp

using namespace kvp;

extern "C" int kvp_trace_generate(const kvp_trace_params* tp, uint32_t* access_bitmaps, void* stream)
{
    if (!tp || !access_bitmaps || !tp->groups || !tp->units_per_group || !tp->steps || (tp->flags & ~KVP_TRACE_SINGLE_PASS))
        return KVP_ERR_ARG;
    if (!tp->topk || tp->topk > tp->units_per_group) return KVP_ERR_ARG;
    if (tp->reserved || (tp->layers > 1 && tp->groups % tp->layers)) return KVP_ERR_ARG;
    if (tp->rho_q < 0 || tp->rho_q > 65536 || tp->c_q < 0 || tp->c_q > (1 << 20) || tp->sigma_q < 0 ||
        tp->sigma_q > (1 << 20))
        return KVP_ERR_ARG;
    const uint64_t U64 = (uint64_t)tp->groups * tp->units_per_group;
    if (U64 >= (1ull << 26) || tp->units_per_group > 8192 || tp->steps > 32768) return KVP_ERR_RANGE;
    // |score| must stay below 2^31: bound |x_t| by its worst case, step by step (|base| <= 2^29 is the caller's)
    {
        const int64_t emax = (((int64_t)262140 * 80265) >> 16) + 1;
        const int64_t jump = tp->burst_thr ? (tp->burst_jump < 0 ? -(int64_t)tp->burst_jump : tp->burst_jump) : 0;
        int64_t bound = (((int64_t)tp->sigma_q * emax) >> 16) + 1 + jump;
        for (uint32_t t = 1; t < tp->steps && bound < (1ll << 30); ++t)
            bound = (((int64_t)tp->rho_q * bound + (int64_t)tp->c_q * emax) >> 16) + 1 + jump;
        if (bound >= (1ll << 30)) return KVP_ERR_RANGE;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    TraceK k;
    k.groups = tp->groups; k.n = tp->units_per_group; k.steps = tp->steps; k.topk = tp->topk;
    k.W32 = (uint32_t)((U64 + 31) / 32);
    k.keys = philox_keys((uint32_t)tp->seed, (uint32_t)(tp->seed >> 32));
    k.rho_q = tp->rho_q; k.c_q = tp->c_q; k.sigma_q = tp->sigma_q; k.burst_jump = tp->burst_jump;
    k.burst_thr = tp->burst_thr; k.base = tp->base; k.out = access_bitmaps;
    k.aligned = tp->units_per_group % 32 == 0;
    k.layers = tp->layers ? tp->layers : 1u;
    k.per_layer = tp->groups / k.layers;
    k.birth = tp->birth;
    const bool layered = k.layers > 1 || k.birth;        // rows of other layers' steps stay zero
    if (!k.aligned || layered) KVP_CUDA(cudaMemsetAsync(access_bitmaps, 0, (size_t)tp->steps * k.W32 * 4, st));
    const uint32_t n = tp->units_per_group;
    const int upt = n <= 1024 ? 1 : n <= 2048 ? 2 : n <= 4096 ? 4 : 8;
    uint32_t T = (n + upt - 1) / upt;
    T = (T + 31) / 32 * 32;
    // Two passes (scores, then one CTA per (group, step)) whenever the score matrix fits a 1 GiB scratch: the work
    // then comes in tens of thousands of equal pieces, while the fused kernel has only `groups` CTAs that walk the
    // steps one after the other (measured: 0.84 vs 0.89 ms on 256 groups of 2048, 1.85 vs 2.11 ms on 640 of 4096,
    // 0.05 vs 2.1 ms on one group of 256).
    const size_t score_bytes = (size_t)U64 * tp->steps * 4;
    if (score_bytes <= ((size_t)1 << 30) && !(tp->flags & KVP_TRACE_SINGLE_PASS) && !layered) {
        int32_t* scores = nullptr;
        int dev = 0;
        KVP_CUDA(cudaGetDevice(&dev));
        int prc = retain_in_pool(dev, score_bytes);          // the next call gets the block back from the pool
        if (prc) return prc;
        KVP_CUDA(cudaMallocAsync(&scores, score_bytes, st));
        if (U64 >= 148u * 1024u) trace_scores_unit_kernel<<<(uint32_t)((U64 + 255) / 256), 256, 0, st>>>(k, (uint32_t)U64, scores);
        else trace_scores_kernel<<<(uint32_t)((U64 + 31) / 32), kScoreThreads, 0, st>>>(k, (uint32_t)U64, scores);
        dim3 grid(tp->groups, tp->steps);
        // Small CTAs with many units per thread: a selection is a chain of barriers and a serial histogram walk, so
        // what counts is how many of them an SM overlaps (whole call, 640 groups of 4096 units x 64 steps: 1.85 ms
        // with 1024 threads, 1.70 ms with 256; 256 groups of 2048 x 128 steps: 0.84 against 0.61 ms with 128). Since the
        // search needs one histogram pass only, eight units per thread are a little faster than sixteen (1.05 against
        // 1.07 ms and 0.359 against 0.363 ms on these two shapes).
        int su = 1;
        while (su < 8 && (n + su - 1) / su > 128) su *= 2;
        const uint32_t ST = ((n + su - 1) / su + 31) / 32 * 32;
        const bool full = (uint64_t)su * ST == n;             // every slot of the CTA holds a unit
#define KVP_SELECT(UPT)                                                                              \
    if (full) trace_select_kernel<UPT, true><<<grid, ST, 0, st>>>(k, (uint32_t)U64, scores);         \
    else trace_select_kernel<UPT, false><<<grid, ST, 0, st>>>(k, (uint32_t)U64, scores)
        switch (su) {
            case 1: KVP_SELECT(1); break;
            case 2: KVP_SELECT(2); break;
            case 4: KVP_SELECT(4); break;
            default: KVP_SELECT(8); break;
        }
#undef KVP_SELECT
        cudaError_t le = cudaGetLastError();
        KVP_CUDA(cudaFreeAsync(scores, st));
        KVP_CUDA(le);
        return KVP_OK;
    }
    if (k.birth) {
        switch (upt) {
            case 1: trace_kernel<1, true><<<tp->groups, T, 0, st>>>(k); break;
            case 2: trace_kernel<2, true><<<tp->groups, T, 0, st>>>(k); break;
            case 4: trace_kernel<4, true><<<tp->groups, T, 0, st>>>(k); break;
            default: trace_kernel<8, true><<<tp->groups, T, 0, st>>>(k); break;
        }
    } else {
        switch (upt) {
            case 1: trace_kernel<1, false><<<tp->groups, T, 0, st>>>(k); break;
            case 2: trace_kernel<2, false><<<tp->groups, T, 0, st>>>(k); break;
            case 4: trace_kernel<4, false><<<tp->groups, T, 0, st>>>(k); break;
            default: trace_kernel<8, false><<<tp->groups, T, 0, st>>>(k); break;
        }
    }
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}
