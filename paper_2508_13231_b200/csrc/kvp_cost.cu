// Cost kernels: per-step cardinalities of a schedule (popc over mask AND placement words) and Eq. 1-5.
//
// The counting pass is the HBM-bound part: every word of A and of P is read once, P[s-1] is carried
// in registers from the previous iteration. Two shapes:
//   wide rows   (>= 17 vectors per row): a warp owns 64 consecutive 16-byte vectors of every row of a
//               step chunk; a CTA of 8 warps therefore reads 8 KB contiguous per row and array.
//   narrow rows (<= 16 vectors per row): a sub-warp group of LPR lanes owns whole rows, consecutive
//               groups own consecutive rows, so a warp still reads contiguous memory.
#include "kvp_common.cuh"

namespace kvp {

namespace {

template <int VEC>
__device__ __forceinline__ uint4 load_vec(const uint32_t* __restrict__ base, size_t row_words, uint32_t row, uint32_t cv)
{
    if (VEC == 4) {
        return __ldg(reinterpret_cast<const uint4*>(base + (size_t)row * row_words) + cv);
    } else {
        return make_uint4(__ldg(base + (size_t)row * row_words + cv), 0u, 0u, 0u);
    }
}

// placement words are read once and never again: stream them through L2 (evict first)
template <int VEC>
__device__ __forceinline__ uint4 load_stream(const uint32_t* __restrict__ base, size_t row_words, uint32_t row, uint32_t cv)
{
    if (VEC == 4) {
        return __ldcs(reinterpret_cast<const uint4*>(base + (size_t)row * row_words) + cv);
    } else {
        return make_uint4(__ldcs(base + (size_t)row * row_words + cv), 0u, 0u, 0u);
    }
}

template <int VEC>
__device__ __forceinline__ uint4 mask_last(uint4 v, uint32_t cv, uint32_t WV, uint32_t pad_mask)
{
    if (cv == WV - 1) {
        if (VEC == 4) v.w &= pad_mask; else v.x &= pad_mask;
    }
    return v;
}

__device__ __forceinline__ uint32_t popc4(uint4 v) { return __popc(v.x) + __popc(v.y) + __popc(v.z) + __popc(v.w); }
__device__ __forceinline__ uint4 and4(uint4 a, uint4 b) { return make_uint4(a.x & b.x, a.y & b.y, a.z & b.z, a.w & b.w); }
__device__ __forceinline__ uint4 andn4(uint4 a, uint4 b) { return make_uint4(a.x & ~b.x, a.y & ~b.y, a.z & ~b.z, a.w & ~b.w); }

// counts of one vector: x = hr | mi << 16, y = mo | occ << 16 (each at most 128)
__device__ __forceinline__ uint2 vec_counts(uint4 a, uint4 p, uint4 prev)
{
    const uint32_t hr = popc4(and4(a, p));
    const uint32_t mi = popc4(andn4(p, prev));
    const uint32_t mo = popc4(andn4(prev, p));
    const uint32_t occ = popc4(p);
    return make_uint2(hr | (mi << 16), mo | (occ << 16));
}

constexpr int WIDE_WARPS = 8;
constexpr int WIDE_VEC = 2;              // 16-byte vectors per lane and row

// Carry-save adder: three bit-vectors in, (carry, sum) out; each bit position is added independently.
__device__ __forceinline__ void csa(uint32_t& carry, uint32_t& sum, uint32_t a, uint32_t b, uint32_t c)
{
    sum = a ^ b ^ c;
    carry = (a & b) | (c & (a ^ b));
}

// Number of set bits in eight words with four popc instead of eight (Harley-Seal): the words are first added
// bit-position-wise into a 4-bit counter held as four bit-vectors. popc is the scarce instruction of this kernel.
__device__ __forceinline__ uint32_t popc8(const uint32_t (&w)[8])
{
    uint32_t ones, twos, fours, eights, ta, tb, tc, td, fa, fb;
    csa(ta, ones, w[0], w[1], w[2]);
    csa(tb, ones, ones, w[3], w[4]);
    csa(tc, ones, ones, w[5], w[6]);
    td = ones & w[7]; ones ^= w[7];
    csa(fa, twos, ta, tb, tc);
    fb = twos & td; twos ^= td;
    eights = fa & fb; fours = fa ^ fb;
    return __popc(ones) + 2 * __popc(twos) + 4 * __popc(fours) + 8 * __popc(eights);
}

// Wide rows: a warp owns 64 consecutive 16-byte vectors (1 KB) of every row of a step chunk, two per lane.
// Per lane and step only three cardinalities are counted, hits |A&P|, occupancy |P| and stayers |P&Pprev|;
// migrations follow as mi = occ - stay and mo = occ_prev - stay.
// GROW (growing cache): L holds the rows of existing units. Placement bits of units that do not exist yet are
// dropped, and the units born in a step (in L[s], not in L[s-1]) that are placed in HBM are a fourth cardinality
// hb: they were written there, not migrated, so mi = occ - stay - hb.
// NS schedules of a batch share a thread: the access words are loaded once and used for all of them, which halves
// the L2 traffic of a batch (A is the half of the bytes that comes from L2, not DRAM).
template <int VEC, bool GROW, int NS>
__global__ void __launch_bounds__(WIDE_WARPS * 32)
count_wide_kernel(const uint32_t* __restrict__ A, const uint32_t* __restrict__ Ps, uint32_t S, uint32_t W32,
                  uint32_t WV, uint32_t pad_mask, uint32_t SC, uint32_t n, uint32_t* __restrict__ counts,
                  const uint32_t* __restrict__ L, uint32_t* __restrict__ hbc)
{
    extern __shared__ uint2 acc[];                       // [NS][WIDE_WARPS][SC], then GROW: uint32 [NS][WIDE_WARPS][SC]
    uint32_t* acc_hb = reinterpret_cast<uint32_t*>(acc + NS * WIDE_WARPS * SC);
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cv0 = (blockIdx.x * WIDE_WARPS + warp) * (32 * WIDE_VEC) + lane;
    const uint32_t sb = blockIdx.y * SC;
    const uint32_t se = min(S, sb + SC);
    const uint32_t* __restrict__ P[NS];
#pragma unroll
    for (int q = 0; q < NS; ++q)                         // a schedule past the batch re-reads the last one; its counts are dropped
        P[q] = Ps + (size_t)min(blockIdx.z * NS + q, n - 1) * S * W32;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    uint4 prev[NS][WIDE_VEC], lprev[WIDE_VEC];
    uint32_t occ_prev[NS];
#pragma unroll
    for (int j = 0; j < WIDE_VEC; ++j) {
        const uint32_t cv = cv0 + 32 * j;
        if (GROW) lprev[j] = cv < WV ? load_vec<VEC>(L, W32, sb ? sb - 1 : 0, cv) : zero;
    }
#pragma unroll
    for (int q = 0; q < NS; ++q) {
        uint32_t w[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
        for (int j = 0; j < WIDE_VEC; ++j) {
            const uint32_t cv = cv0 + 32 * j;
            prev[q][j] = cv < WV ? mask_last<VEC>(load_vec<VEC>(P[q], W32, sb ? sb - 1 : 0, cv), cv, WV, pad_mask) : zero;
            if (GROW) prev[q][j] = and4(prev[q][j], lprev[j]);
            w[4 * j] = prev[q][j].x; w[4 * j + 1] = prev[q][j].y; w[4 * j + 2] = prev[q][j].z; w[4 * j + 3] = prev[q][j].w;
        }
        occ_prev[q] = popc8(w);
    }
#pragma unroll 4
    for (uint32_t s = sb; s < se; ++s) {
        uint4 a[WIDE_VEC], l[WIDE_VEC], p[NS][WIDE_VEC];
#pragma unroll
        for (int j = 0; j < WIDE_VEC; ++j) {
            const uint32_t cv = cv0 + 32 * j;
            const bool valid = cv < WV;
            a[j] = valid ? load_vec<VEC>(A, W32, s, cv) : zero;
            if (GROW) l[j] = valid ? load_vec<VEC>(L, W32, s, cv) : zero;
#pragma unroll
            for (int q = 0; q < NS; ++q)
                p[q][j] = valid ? mask_last<VEC>(load_stream<VEC>(P[q], W32, s, cv), cv, WV, pad_mask) : zero;
        }
#pragma unroll
        for (int q = 0; q < NS; ++q) {
            uint32_t wp[8], wh[8], ws[8], wb[8];
#pragma unroll
            for (int j = 0; j < WIDE_VEC; ++j) {
                uint4 pj = p[q][j];
                if (GROW) {
                    pj = and4(pj, l[j]);
                    const uint4 born = andn4(pj, lprev[j]);          // placed in HBM in the step it is written
                    wb[4 * j] = born.x; wb[4 * j + 1] = born.y; wb[4 * j + 2] = born.z; wb[4 * j + 3] = born.w;
                }
                wp[4 * j] = pj.x; wp[4 * j + 1] = pj.y; wp[4 * j + 2] = pj.z; wp[4 * j + 3] = pj.w;
                wh[4 * j] = a[j].x & pj.x; wh[4 * j + 1] = a[j].y & pj.y;
                wh[4 * j + 2] = a[j].z & pj.z; wh[4 * j + 3] = a[j].w & pj.w;
                ws[4 * j] = pj.x & prev[q][j].x; ws[4 * j + 1] = pj.y & prev[q][j].y;
                ws[4 * j + 2] = pj.z & prev[q][j].z; ws[4 * j + 3] = pj.w & prev[q][j].w;
                prev[q][j] = pj;
            }
            const uint32_t occ = popc8(wp), hr = popc8(wh), stay = popc8(ws);
            uint32_t hb = 0;
            if (GROW) hb = popc8(wb);
            uint2 c = make_uint2(hr | ((occ - stay - hb) << 16), (occ_prev[q] - stay) | (occ << 16));
            occ_prev[q] = occ;
            c.x = __reduce_add_sync(0xFFFFFFFFu, c.x);   // 16-bit fields: 32 lanes * 256 < 65536
            c.y = __reduce_add_sync(0xFFFFFFFFu, c.y);
            if (GROW) hb = __reduce_add_sync(0xFFFFFFFFu, hb);
            if (lane == 0) {
                acc[(q * WIDE_WARPS + warp) * SC + (s - sb)] = c;
                if (GROW) acc_hb[(q * WIDE_WARPS + warp) * SC + (s - sb)] = hb;
            }
        }
        if (GROW) {
#pragma unroll
            for (int j = 0; j < WIDE_VEC; ++j) lprev[j] = l[j];
        }
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < NS; ++q) {
        const uint32_t sched = blockIdx.z * NS + q;
        if (sched >= n) break;
        for (uint32_t i = threadIdx.x; i < se - sb; i += blockDim.x) {
            uint32_t hr = 0, mi = 0, mo = 0, occ = 0;
#pragma unroll
            for (int w = 0; w < WIDE_WARPS; ++w) {
                const uint2 c = acc[(q * WIDE_WARPS + w) * SC + i];
                hr += c.x & 0xFFFFu; mi += c.x >> 16; mo += c.y & 0xFFFFu; occ += c.y >> 16;
            }
            uint32_t* dst = counts + ((size_t)sched * S + sb + i) * 4;
            if (hr) atomicAdd(dst + 0, hr);
            if (mi) atomicAdd(dst + 1, mi);
            if (mo) atomicAdd(dst + 2, mo);
            if (occ) atomicAdd(dst + 3, occ);
            if (GROW) {
                uint32_t hb = 0;
#pragma unroll
                for (int w = 0; w < WIDE_WARPS; ++w) hb += acc_hb[(q * WIDE_WARPS + w) * SC + i];
                if (hb) atomicAdd(hbc + (size_t)sched * S + sb + i, hb);
            }
        }
    }
}

constexpr int NARROW_ITERS = 8;

template <int VEC, int LPR, bool GROW>
__global__ void __launch_bounds__(256)
count_narrow_kernel(const uint32_t* __restrict__ A, const uint32_t* __restrict__ Ps, uint32_t S, uint32_t W32,
                    uint32_t WV, uint32_t pad_mask, uint32_t* __restrict__ counts, const uint32_t* __restrict__ L,
                    uint32_t* __restrict__ hbc)
{
    constexpr uint32_t GROUPS = 256 / LPR;               // rows in flight per CTA
    const uint32_t g = threadIdx.x / LPR, cv = threadIdx.x % LPR;
    const bool col_ok = cv < WV;
    const uint32_t* __restrict__ P = Ps + (size_t)blockIdx.y * S * W32;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 2
    for (int it = 0; it < NARROW_ITERS; ++it) {
        const uint32_t s = (blockIdx.x * NARROW_ITERS + it) * GROUPS + g;
        const bool ok = col_ok && s < S;
        const uint4 a = ok ? load_vec<VEC>(A, W32, s, cv) : zero;
        uint4 p = ok ? mask_last<VEC>(load_vec<VEC>(P, W32, s, cv), cv, WV, pad_mask) : zero;
        uint4 q = ok ? mask_last<VEC>(load_vec<VEC>(P, W32, s ? s - 1 : 0, cv), cv, WV, pad_mask) : zero;
        uint32_t hb = 0;
        if (GROW) {                                      // see count_wide_kernel
            const uint4 l = ok ? load_vec<VEC>(L, W32, s, cv) : zero;
            const uint4 lq = ok ? load_vec<VEC>(L, W32, s ? s - 1 : 0, cv) : zero;
            p = and4(p, l);
            q = and4(q, lq);
            hb = popc4(andn4(p, lq));
        }
        uint2 c = vec_counts(a, p, q);
        if (GROW) c.x -= hb << 16;                       // born in HBM: written, not migrated in
#pragma unroll
        for (int off = LPR / 2; off > 0; off >>= 1) {
            c.x += __shfl_xor_sync(0xFFFFFFFFu, c.x, off);
            c.y += __shfl_xor_sync(0xFFFFFFFFu, c.y, off);
            if (GROW) hb += __shfl_xor_sync(0xFFFFFFFFu, hb, off);
        }
        if (cv == 0 && s < S) {
            reinterpret_cast<uint4*>(counts)[(size_t)blockIdx.y * S + s] =
                make_uint4(c.x & 0xFFFFu, c.x >> 16, c.y & 0xFFFFu, c.y >> 16);
            if (GROW) hbc[(size_t)blockIdx.y * S + s] = hb;
        }
    }
}

__global__ void __launch_bounds__(256)
finish_kernel(const uint4* __restrict__ counts, const uint32_t* __restrict__ hbc, const StepC* __restrict__ stepc, CostK K,
              uint32_t S, uint32_t cap,
              double spt, uint64_t* __restrict__ step_ticks, uint64_t* __restrict__ total_ticks,
              double* __restrict__ step_seconds, double* __restrict__ total_seconds, int32_t* __restrict__ bad_step,
              uint64_t* __restrict__ hits)
{
    __shared__ uint64_t s_sum[8], s_hit[8];
    __shared__ uint32_t s_bad[8];
    const uint32_t i = blockIdx.x;
    uint64_t sum = 0, hit = 0;
    uint32_t bad = 0xFFFFFFFFu;
    for (uint32_t s = threadIdx.x; s < S; s += blockDim.x) {
        const uint4 c = counts[(size_t)i * S + s];
        const uint32_t f = hbc ? step_cost_g(c.x, c.y, c.z, hbc[(size_t)i * S + s], __ldg(&stepc[s]), K)
                               : step_cost(c.x, c.y, c.z, __ldg(&stepc[s]), K);
        if (step_ticks) step_ticks[(size_t)i * S + s] = f;
        if (step_seconds) step_seconds[(size_t)i * S + s] = (double)f * spt;
        sum += f;
        hit += c.x;
        if (c.w > cap) bad = min(bad, s);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        sum += __shfl_xor_sync(0xFFFFFFFFu, sum, off);
        hit += __shfl_xor_sync(0xFFFFFFFFu, hit, off);
        bad = min(bad, __shfl_xor_sync(0xFFFFFFFFu, bad, off));
    }
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { s_sum[warp] = sum; s_hit[warp] = hit; s_bad[warp] = bad; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) { sum += s_sum[w]; hit += s_hit[w]; bad = min(bad, s_bad[w]); }
        if (total_ticks) total_ticks[i] = sum;
        if (total_seconds) total_seconds[i] = (double)sum * spt;
        if (bad_step) bad_step[i] = bad == 0xFFFFFFFFu ? -1 : (int32_t)bad;
        if (hits) hits[i] = hit;
    }
}

__global__ void __launch_bounds__(256)
row_popcount_kernel(const uint32_t* __restrict__ rows, uint32_t S, uint32_t W32, uint32_t* __restrict__ out)
{
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= S) return;
    uint32_t c = 0;
    for (uint32_t w = lane; w < W32; w += 32) c += __popc(__ldg(rows + (size_t)warp * W32 + w));
    c = __reduce_add_sync(0xFFFFFFFFu, c);
    if (lane == 0) out[warp] = c;
}

template <int VEC, bool GROW>
int launch_narrow(uint32_t WV, uint32_t n, const uint32_t* A, const uint32_t* P, uint32_t S, uint32_t W32,
                  uint32_t pad_mask, uint32_t* counts, const uint32_t* L, uint32_t* hbc, cudaStream_t st)
{
#define KVP_NARROW(LPR)                                                                                          \
    {                                                                                                            \
        const uint32_t rows_per_cta = (256 / LPR) * NARROW_ITERS;                                                \
        dim3 grid((S + rows_per_cta - 1) / rows_per_cta, n);                                                     \
        count_narrow_kernel<VEC, LPR, GROW><<<grid, 256, 0, st>>>(A, P, S, W32, WV, pad_mask, counts, L, hbc);   \
    }
    if (WV <= 1) KVP_NARROW(1)
    else if (WV <= 2) KVP_NARROW(2)
    else if (WV <= 4) KVP_NARROW(4)
    else if (WV <= 8) KVP_NARROW(8)
    else KVP_NARROW(16)
#undef KVP_NARROW
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

}  // namespace

int launch_row_popcount(const uint32_t* rows, uint32_t S, uint32_t W32, uint32_t* out, cudaStream_t st)
{
    row_popcount_kernel<<<(S + 7) / 8, 256, 0, st>>>(rows, S, W32, out);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

// counts [n][S][4] = {hr, mi, mo, occ}; hbc [n][S] for a problem with births
int launch_counts(const kvp_problem* p, const uint32_t* schedules, uint32_t n, uint32_t* counts, uint32_t* hbc,
                  cudaStream_t st, uint32_t* launches)
{
    const bool grow = p->dL != nullptr;
    if (grow && !hbc) return KVP_ERR_ARG;
    const bool vec4 = (p->W32 % 4 == 0) && ((reinterpret_cast<uintptr_t>(schedules) & 15) == 0);
    const uint32_t WV = vec4 ? p->W32 / 4 : p->W32;
    if (WV <= 16) {
        if (launches) *launches += 1;
        if (grow)
            return vec4 ? launch_narrow<4, true>(WV, n, p->dA, schedules, p->S, p->W32, p->pad_mask, counts, p->dL, hbc, st)
                        : launch_narrow<1, true>(WV, n, p->dA, schedules, p->S, p->W32, p->pad_mask, counts, p->dL, hbc, st);
        return vec4 ? launch_narrow<4, false>(WV, n, p->dA, schedules, p->S, p->W32, p->pad_mask, counts, nullptr, nullptr, st)
                    : launch_narrow<1, false>(WV, n, p->dA, schedules, p->S, p->W32, p->pad_mask, counts, nullptr, nullptr, st);
    }
    KVP_CUDA(cudaMemsetAsync(counts, 0, (size_t)n * p->S * 16, st));
    if (grow) KVP_CUDA(cudaMemsetAsync(hbc, 0, (size_t)n * p->S * 4, st));
    const uint32_t col_ctas = (WV + WIDE_WARPS * 32 * WIDE_VEC - 1) / (WIDE_WARPS * 32 * WIDE_VEC);
    // two schedules per thread once a batch is large enough to fill the GPU that way
    const uint32_t NS = n >= 8 ? 2u : 1u;
    const uint32_t nz = (n + NS - 1) / NS;
    // Split the steps until the grid is at least four full waves (148 SMs x 8 resident CTAs), so that the last,
    // partial wave costs little; every chunk re-reads one halo row (1/SC more traffic, mostly from L2).
    uint32_t SC = p->S;
    while (SC > 8 && (uint64_t)col_ctas * ((p->S + SC - 1) / SC) * nz < 148u * 8u * 4u) SC = (SC + 1) / 2;
    // the per-step accumulators of a chunk live in dynamic shared memory: keep them within the 48 KB a kernel gets
    // without opting in (NS * WIDE_WARPS * SC entries of 8 bytes, 12 with births)
    const uint32_t sc_max = (uint32_t)((48u * 1024u) / (NS * WIDE_WARPS * (sizeof(uint2) + (grow ? 4 : 0))));
    if (SC > sc_max) SC = sc_max;
    dim3 grid(col_ctas, (p->S + SC - 1) / SC, nz);
    const size_t smem = (size_t)NS * WIDE_WARPS * SC * (sizeof(uint2) + (grow ? 4 : 0));
    const int T = WIDE_WARPS * 32;
#define KVP_WIDE(VEC, GROW, NSCH)                                                                                  \
    count_wide_kernel<VEC, GROW, NSCH><<<grid, T, smem, st>>>(p->dA, schedules, p->S, p->W32, WV, p->pad_mask, SC, n, \
                                                              counts, GROW ? p->dL : nullptr, GROW ? hbc : nullptr)
    if (NS == 2) {
        if (grow) { if (vec4) KVP_WIDE(4, true, 2); else KVP_WIDE(1, true, 2); }
        else { if (vec4) KVP_WIDE(4, false, 2); else KVP_WIDE(1, false, 2); }
    } else {
        if (grow) { if (vec4) KVP_WIDE(4, true, 1); else KVP_WIDE(1, true, 1); }
        else { if (vec4) KVP_WIDE(4, false, 1); else KVP_WIDE(1, false, 1); }
    }
#undef KVP_WIDE
    KVP_CUDA(cudaGetLastError());
    if (launches) *launches += 1;
    return KVP_OK;
}

int launch_finish(const kvp_problem* p, const uint32_t* counts, const uint32_t* hbc, uint32_t n, uint64_t* step_ticks,
                  uint64_t* total_ticks, double* step_seconds, double* total_seconds, int32_t* bad_step, uint64_t* hits,
                  cudaStream_t st)
{
    if (p->dL && !hbc) return KVP_ERR_ARG;
    finish_kernel<<<n, 256, 0, st>>>(reinterpret_cast<const uint4*>(counts), p->dL ? hbc : nullptr, p->d_stepc, p->K, p->S,
                                      p->cap, p->spt, step_ticks, total_ticks, step_seconds, total_seconds, bad_step, hits);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

}  // namespace kvp

// The schedule index is a grid dimension limited to 65535: larger batches go in slices.
static const uint32_t kBatchSlice = 32768;

extern "C" int kvp_eval_counts(kvp_problem* p, const uint32_t* schedules, uint32_t n, uint32_t* counts, void* stream)
{
    if (!p || !schedules || !counts || !n) return KVP_ERR_ARG;
    if (p->dL) return KVP_ERR_ARG;                       // four cardinalities do not describe a growing cache
    if ((reinterpret_cast<uintptr_t>(counts) & 15) != 0) return KVP_ERR_ARG;
    KVP_CUDA(cudaSetDevice(p->device));
    p->last_stream = static_cast<cudaStream_t>(stream);
    const size_t sched_words = (size_t)p->S * p->W32;
    for (uint32_t i = 0; i < n; i += kBatchSlice) {
        const uint32_t m = n - i < kBatchSlice ? n - i : kBatchSlice;
        int rc = kvp::launch_counts(p, schedules + i * sched_words, m, counts + (size_t)i * p->S * 4, nullptr,
                                    static_cast<cudaStream_t>(stream), nullptr);
        if (rc) return rc;
    }
    return KVP_OK;
}

extern "C" int kvp_eval(kvp_problem* p, const uint32_t* schedules, uint32_t n, uint64_t* step_ticks, uint64_t* total_ticks,
                        double* step_seconds, double* total_seconds, int32_t* bad_step, void* stream)
{
    if (!p || !schedules || !total_ticks || !n) return KVP_ERR_ARG;
    KVP_CUDA(cudaSetDevice(p->device));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint32_t slice = n < kBatchSlice ? n : kBatchSlice;
    int rc = kvp::ensure_scratch(p, (size_t)slice * p->S * 20, st);
    if (rc) return rc;
    uint32_t* counts = static_cast<uint32_t*>(p->d_scratch);
    uint32_t* hbc = counts + (size_t)slice * p->S * 4;   // used by problems with births only
    const size_t sched_words = (size_t)p->S * p->W32;
    for (uint32_t i = 0; i < n; i += kBatchSlice) {
        const uint32_t m = n - i < kBatchSlice ? n - i : kBatchSlice;
        if ((rc = kvp::launch_counts(p, schedules + i * sched_words, m, counts, hbc, st, nullptr))) return rc;
        const size_t so = (size_t)i * p->S;
        if ((rc = kvp::launch_finish(p, counts, hbc, m, step_ticks ? step_ticks + so : nullptr, total_ticks + i,
                                     step_seconds ? step_seconds + so : nullptr,
                                     total_seconds ? total_seconds + i : nullptr, bad_step ? bad_step + i : nullptr,
                                     nullptr, st)))
            return rc;
    }
    return KVP_OK;
}

// ---------------------------------------------------------------------------------------------------
// kvp_eval without any allocation: the per-step cardinalities go to a fixed array in the library image.
// Meant for callers that cannot afford or are not allowed a cudaMalloc at this point (a latency-bound
// loop, a process whose memory pool owns the whole device, allocator-free code). See include/kvp.h.
static __device__ __align__(256) uint32_t g_noalloc_counts[KVP_NOALLOC_SCRATCH_BYTES / 4];

namespace {
constexpr int kMaxDevices = 64;
uint32_t* g_noalloc_addr[kMaxDevices];   // device address of g_noalloc_counts, per device; null until looked up
}

// In host code `g_noalloc_counts` names a host-side shadow of the symbol, not device memory: the address a
// kernel may use has to be asked for, once per device and with that device current.
static int noalloc_scratch(int device, uint32_t** out)
{
    if (device < 0 || device >= kMaxDevices) return KVP_ERR_RANGE;
    uint32_t* ptr = __atomic_load_n(&g_noalloc_addr[device], __ATOMIC_ACQUIRE);
    if (!ptr) {
        KVP_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_counts));
        if (!ptr) return KVP_ERR_CUDA;
        __atomic_store_n(&g_noalloc_addr[device], ptr, __ATOMIC_RELEASE);   // racing threads store the same value
    }
    *out = ptr;
    return KVP_OK;
}

extern "C" int kvp_eval_noalloc(kvp_problem* p, const uint32_t* schedules, uint32_t n, uint64_t* step_ticks,
                                uint64_t* total_ticks, double* step_seconds, double* total_seconds, int32_t* bad_step,
                                void* stream)
{
    if (!p || !schedules || !total_ticks || !n || p->dL) return KVP_ERR_ARG;
    if ((uint64_t)n * p->S * 16ull > (uint64_t)KVP_NOALLOC_SCRATCH_BYTES) return KVP_ERR_RANGE;   // batch too large
    KVP_CUDA(cudaSetDevice(p->device));
    uint32_t* counts = nullptr;
    int rc = noalloc_scratch(p->device, &counts);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    // The array still holds the previous call's numbers. launch_counts either overwrites every entry it
    // owns (narrow rows) or clears them on the stream before accumulating (wide rows). The schedule index is a
    // grid dimension, so a batch of more than kBatchSlice schedules (possible within the limit only for one or two
    // steps) goes in slices, each with its own part of the array.
    const size_t sched_words = (size_t)p->S * p->W32;
    for (uint32_t i = 0; i < n; i += kBatchSlice) {
        const uint32_t m = n - i < kBatchSlice ? n - i : kBatchSlice;
        const size_t so = (size_t)i * p->S;
        uint32_t* part = counts + so * 4;
        if ((rc = kvp::launch_counts(p, schedules + i * sched_words, m, part, nullptr, st, nullptr))) return rc;
        if ((rc = kvp::launch_finish(p, part, nullptr, m, step_ticks ? step_ticks + so : nullptr, total_ticks + i,
                                     step_seconds ? step_seconds + so : nullptr,
                                     total_seconds ? total_seconds + i : nullptr, bad_step ? bad_step + i : nullptr,
                                     nullptr, st)))
            return rc;
    }
    return KVP_OK;
}
