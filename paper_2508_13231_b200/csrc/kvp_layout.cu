// Layout kernels: bit-matrix transposes between the step-major API layout and the time-packed layout
// the annealer works on, pad-bit cleaning, per-unit access counts and the static initial placements.
#include "kvp_common.cuh"

namespace kvp {

namespace {

// in: [rows][in_words] words, bit c of row r = bit (c & 31) of in[r][c >> 5].
// out: [cols][out_words], bit r of row c. Bits beyond `rows` in the last out word are 0.
// One CTA transposes a tile of 32 rows x 32 words (1024 columns); warp w owns word column w.
__global__ void __launch_bounds__(1024)
bit_transpose_kernel(const uint32_t* __restrict__ in, uint32_t rows, uint32_t in_words, uint32_t cols,
                     uint32_t* __restrict__ out, uint32_t out_words)
{
    __shared__ uint32_t tile[32][33];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t r0 = blockIdx.x * 32, w0 = blockIdx.y * 32;   // row blocks can be millions: they go in x
    // coalesced load: warp `warp` reads row r0 + warp, lanes read consecutive words
    {
        const uint32_t r = r0 + warp, w = w0 + lane;
        tile[warp][lane] = (r < rows && w < in_words) ? __ldg(in + (size_t)r * in_words + w) : 0u;
    }
    __syncthreads();
    // warp `warp` now transposes word column w0 + warp: lane l holds row r0 + l
    const uint32_t word = tile[lane][warp];
    uint32_t mine = 0;
#pragma unroll
    for (int b = 0; b < 32; ++b) {
        const uint32_t col_bits = __ballot_sync(0xFFFFFFFFu, (word >> b) & 1u);
        if (lane == (uint32_t)b) mine = col_bits;
    }
    const uint32_t c = (w0 + warp) * 32 + lane;
    if (c < cols) out[(size_t)c * out_words + blockIdx.x] = mine;
}

__global__ void clean_copy_kernel(const uint32_t* __restrict__ in, uint32_t* __restrict__ out, size_t total,
                                  uint32_t W32, uint32_t pad_mask)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        uint32_t v = in[i];
        if (i % W32 == W32 - 1) v &= pad_mask;
        out[i] = v;
    }
}

__global__ void unit_counts_kernel(const uint32_t* __restrict__ Acol, uint32_t U, uint32_t S32, uint32_t* __restrict__ ucnt)
{
    const uint32_t u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= U) return;
    uint32_t c = 0;
    for (uint32_t j = 0; j < S32; ++j) c += __popc(__ldg(Acol + (size_t)u * S32 + j));
    ucnt[u] = c;
}

// Histogram of the per-unit access counts (bins 0..S). Few bins and millions of units: every CTA counts its units in
// shared memory first (when the bins fit) and adds only its non-empty bins to the global histogram.
constexpr uint32_t kHistBins = 8192;
__global__ void __launch_bounds__(1024)
histogram_kernel(const uint32_t* __restrict__ ucnt, uint32_t U, uint32_t bins, uint32_t* __restrict__ hist)
{
    __shared__ uint32_t local[kHistBins];
    const bool staged = bins <= kHistBins;
    if (staged) {
        for (uint32_t b = threadIdx.x; b < bins; b += blockDim.x) local[b] = 0u;
        __syncthreads();
    }
    for (uint32_t u = blockIdx.x * blockDim.x + threadIdx.x; u < U; u += gridDim.x * blockDim.x)
        atomicAdd((staged ? local : hist) + ucnt[u], 1u);
    if (staged) {
        __syncthreads();
        for (uint32_t b = threadIdx.x; b < bins; b += blockDim.x)
            if (local[b]) atomicAdd(hist + b, local[b]);
    }
}

// The `cap` most accessed units, ties to the lower index, in three steps. First, one CTA finds the count threshold
// from the histogram: sel = {threshold count, number of ties to take}.
__global__ void __launch_bounds__(1024)
static_threshold_kernel(const uint32_t* __restrict__ hist, uint32_t S, uint32_t cap, uint32_t* __restrict__ sel)
{
    __shared__ uint32_t s_thr, s_take, s_found;
    __shared__ uint32_t s_warp[32];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { s_thr = S + 1; s_take = 0; s_found = 0; }
    __syncthreads();
    // counts run 0..S; descend, 1024 counts at a time (thread i looks at count top - i), until the capacity is reached
    if (cap != 0) {
        uint32_t above = 0;                               // units with a count above this chunk
        for (int64_t top = S; top >= 0; top -= 1024) {
            const int64_t c = top - (int64_t)threadIdx.x;
            const uint32_t h = c >= 0 ? hist[c] : 0u;
            uint32_t incl = h;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= (uint32_t)off) incl += v;
            }
            if (lane == 31) s_warp[warp] = incl;
            __syncthreads();
            uint32_t before = 0, total = 0;
            for (uint32_t w = 0; w < 32; ++w) {
                const uint32_t v = s_warp[w];
                before += w < warp ? v : 0u;
                total += v;
            }
            incl += before + above;
            const uint32_t excl = incl - h;
            if (c >= 0 && excl < cap && incl >= cap) { s_thr = (uint32_t)c; s_take = cap - excl; s_found = 1; }   // one thread at most
            __syncthreads();
            if (s_found) break;
            above += total;
            __syncthreads();
        }
    }
    if (threadIdx.x == 0) { sel[0] = s_thr; sel[1] = s_take; }
}

// Second, every CTA counts the ties (units whose count equals the threshold) among its 1024 units.
__global__ void __launch_bounds__(1024)
static_ties_kernel(const uint32_t* __restrict__ ucnt, const uint32_t* __restrict__ sel, uint32_t U, uint32_t* __restrict__ ties)
{
    const uint32_t u = blockIdx.x * 1024 + threadIdx.x;
    const int n = __syncthreads_count(u < U && ucnt[u] == sel[0]);
    if (threadIdx.x == 0) ties[blockIdx.x] = (uint32_t)n;
}

// Third, every CTA takes its units above the threshold and as many of its ties as are left after the ties of the CTAs
// before it (ties go to the lower index).
__global__ void __launch_bounds__(1024)
static_pick_kernel(const uint32_t* __restrict__ ucnt, const uint32_t* __restrict__ sel, const uint32_t* __restrict__ ties,
                   uint32_t U, uint32_t* __restrict__ row, uint32_t W32)
{
    __shared__ uint32_t s_warp[32];
    __shared__ uint32_t s_base;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t thr = sel[0], take = sel[1];
    uint32_t mine = 0;
    for (uint32_t j = threadIdx.x; j < blockIdx.x; j += 1024) mine += ties[j];
    mine = __reduce_add_sync(0xFFFFFFFFu, mine);
    if (lane == 0) s_warp[warp] = mine;
    __syncthreads();
    if (threadIdx.x == 0) { uint32_t t = 0; for (int w = 0; w < 32; ++w) t += s_warp[w]; s_base = t; }
    __syncthreads();
    const uint32_t base = s_base;
    __syncthreads();
    const uint32_t u = blockIdx.x * 1024 + threadIdx.x;
    const uint32_t c = u < U ? ucnt[u] : 0xFFFFFFFFu;
    const bool tie = u < U && c == thr;
    const uint32_t tie_bits = __ballot_sync(0xFFFFFFFFu, tie);
    if (lane == 0) s_warp[warp] = __popc(tie_bits);
    __syncthreads();
    uint32_t before = base;
    for (uint32_t w = 0; w < warp; ++w) before += s_warp[w];
    before += __popc(tie_bits & ((1u << lane) - 1u));
    const bool pick = u < U && (c > thr || (tie && before < take));
    const uint32_t bits = __ballot_sync(0xFFFFFFFFu, pick);
    if (lane == 0 && u < W32 * 32) row[u >> 5] = bits;
}

__global__ void static_first_kernel(uint32_t* __restrict__ row, uint32_t W32, uint32_t cap)
{
    const uint32_t w = blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= W32) return;
    const uint32_t lo = w * 32;
    row[w] = cap >= lo + 32 ? 0xFFFFFFFFu : (cap > lo ? (1u << (cap - lo)) - 1u : 0u);
}

__global__ void broadcast_row_kernel(const uint32_t* __restrict__ row, uint32_t W32, size_t total, uint32_t* __restrict__ sched)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x)
        sched[i] = __ldg(row + i % W32);
}

// time-packed columns of a schedule whose every row equals `row`
__global__ void row_to_columns_kernel(const uint32_t* __restrict__ row, uint32_t U, uint32_t S, uint32_t S32,
                                      uint32_t* __restrict__ Pcol)
{
    const size_t total = (size_t)U * S32;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const uint32_t u = (uint32_t)(i / S32), j = (uint32_t)(i % S32);
        const uint32_t on = (__ldg(row + (u >> 5)) >> (u & 31)) & 1u;
        const uint32_t valid = (j + 1) * 32 <= S ? 0xFFFFFFFFu : ((1u << (S - j * 32)) - 1u);
        Pcol[i] = on ? valid : 0u;
    }
}

// Growing cache: row s of L has bit u set iff unit u exists at step s (birth[u] <= s). One thread per word.
__global__ void alive_rows_kernel(const uint32_t* __restrict__ birth, uint32_t U, uint32_t W32, size_t total,
                                  uint32_t* __restrict__ L)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const uint32_t s = (uint32_t)(i / W32), u0 = (uint32_t)(i % W32) * 32;
        uint32_t bits = 0;
        for (uint32_t b = 0; b < 32 && u0 + b < U; ++b) bits |= (__ldg(birth + u0 + b) <= s ? 1u : 0u) << b;
        L[i] = bits;
    }
}

// Births per step, and the checks of kvp_set_births: flag bit 0 = a birth beyond the horizon, bit 1 = a unit
// that is accessed before it exists.
__global__ void birth_stats_kernel(const uint32_t* __restrict__ birth, uint32_t U, uint32_t S,
                                   const uint32_t* __restrict__ Acol, uint32_t S32, uint32_t* __restrict__ nb,
                                   uint32_t* __restrict__ flag)
{
    const uint32_t u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= U) return;
    const uint32_t b = birth[u];
    if (b >= S) { atomicOr(flag, 1u); return; }
    if (b == 0) return;
    atomicAdd(nb + b, 1u);
    uint32_t early = 0;
    for (uint32_t j = 0; j < (b >> 5); ++j) early |= __ldg(Acol + (size_t)u * S32 + j);
    if (b & 31u) early |= __ldg(Acol + (size_t)u * S32 + (b >> 5)) & ((1u << (b & 31u)) - 1u);
    if (early) atomicOr(flag, 2u);
}

// every unit born in a step is first counted as written to DRAM (see step_cost_g)
__global__ void stepc_births_kernel(StepC* __restrict__ stepc, const uint32_t* __restrict__ nb, uint32_t S, uint32_t kk,
                                    uint32_t kd)
{
    const uint32_t s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= S) return;
    StepC c = stepc[s];
    c.y += kk * nb[s];
    c.z += kd * nb[s];
    stepc[s] = c;
}

__global__ void and_rows_kernel(uint32_t* __restrict__ sched, const uint32_t* __restrict__ L, size_t total)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x)
        sched[i] &= __ldg(L + i);
}

inline uint32_t grid_for(size_t total, uint32_t block)
{
    size_t g = (total + block - 1) / block;
    return (uint32_t)(g > 148 * 16 ? 148 * 16 : (g ? g : 1));
}

}  // namespace

int launch_bit_transpose(const uint32_t* in, uint32_t rows, uint32_t in_words, uint32_t cols, uint32_t* out,
                         uint32_t out_words, cudaStream_t st)
{
    dim3 grid((rows + 31) / 32, (in_words + 31) / 32);
    bit_transpose_kernel<<<grid, 1024, 0, st>>>(in, rows, in_words, cols, out, out_words);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

int launch_clean_copy(const uint32_t* in, uint32_t* out, uint32_t S, uint32_t W32, uint32_t pad_mask, cudaStream_t st)
{
    const size_t total = (size_t)S * W32;
    clean_copy_kernel<<<grid_for(total, 256), 256, 0, st>>>(in, out, total, W32, pad_mask);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

int launch_unit_counts(const uint32_t* Acol, uint32_t U, uint32_t S32, uint32_t* ucnt, cudaStream_t st)
{
    unit_counts_kernel<<<(U + 255) / 256, 256, 0, st>>>(Acol, U, S32, ucnt);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

// needs (S + 1) * 4 bytes of zeroed scratch for the histogram; uses p->d_scratch
int launch_static_freq_row(const kvp_problem* p, uint32_t* row, cudaStream_t st)
{
    // scratch: the histogram (S + 1 bins), the selection (2 words), the tie counts of the chunks of 1024 units
    uint32_t* hist = static_cast<uint32_t*>(p->d_scratch);
    uint32_t* sel = hist + ((p->S + 1 + 3) & ~3u);
    uint32_t* ties = sel + 4;
    const uint32_t chunks = (p->W32 * 32 + 1023) / 1024;
    KVP_CUDA(cudaMemsetAsync(hist, 0, (size_t)(p->S + 1) * 4, st));
    uint32_t hgrid = (p->U + 16383) / 16384;
    if (hgrid > 1184) hgrid = 1184;
    histogram_kernel<<<hgrid, 1024, 0, st>>>(p->d_ucnt, p->U, p->S + 1, hist);
    KVP_CUDA(cudaGetLastError());
    static_threshold_kernel<<<1, 1024, 0, st>>>(hist, p->S, p->cap, sel);
    KVP_CUDA(cudaGetLastError());
    static_ties_kernel<<<chunks, 1024, 0, st>>>(p->d_ucnt, sel, p->U, ties);
    KVP_CUDA(cudaGetLastError());
    static_pick_kernel<<<chunks, 1024, 0, st>>>(p->d_ucnt, sel, ties, p->U, row, p->W32);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

int launch_static_first_row(const kvp_problem* p, uint32_t* row, cudaStream_t st)
{
    static_first_kernel<<<(p->W32 + 255) / 256, 256, 0, st>>>(row, p->W32, p->cap);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

int launch_broadcast_row(const uint32_t* row, uint32_t S, uint32_t W32, uint32_t* sched, cudaStream_t st)
{
    const size_t total = (size_t)S * W32;
    broadcast_row_kernel<<<grid_for(total, 256), 256, 0, st>>>(row, W32, total, sched);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

int launch_row_to_columns(const uint32_t* row, uint32_t U, uint32_t S, uint32_t S32, uint32_t* Pcol, cudaStream_t st)
{
    const size_t total = (size_t)U * S32;
    row_to_columns_kernel<<<grid_for(total, 256), 256, 0, st>>>(row, U, S, S32, Pcol);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

int launch_alive_rows(const uint32_t* birth, uint32_t U, uint32_t S, uint32_t W32, uint32_t* L, cudaStream_t st)
{
    const size_t total = (size_t)S * W32;
    alive_rows_kernel<<<grid_for(total, 256), 256, 0, st>>>(birth, U, W32, total, L);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

int launch_birth_stats(const uint32_t* birth, uint32_t U, uint32_t S, const uint32_t* Acol, uint32_t S32, uint32_t* nb,
                       uint32_t* flag, cudaStream_t st)
{
    birth_stats_kernel<<<(U + 255) / 256, 256, 0, st>>>(birth, U, S, Acol, S32, nb, flag);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

int launch_stepc_births(StepC* stepc, const uint32_t* nb, uint32_t S, uint32_t kk, uint32_t kd, cudaStream_t st)
{
    stepc_births_kernel<<<(S + 255) / 256, 256, 0, st>>>(stepc, nb, S, kk, kd);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

int launch_and_rows(uint32_t* sched, const uint32_t* L, size_t total, cudaStream_t st)
{
    and_rows_kernel<<<grid_for(total, 256), 256, 0, st>>>(sched, L, total);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

}  // namespace kvp
