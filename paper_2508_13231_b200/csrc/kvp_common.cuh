// Shared declarations of the CUDA implementation of include/kvp.h (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/kvp.h"

namespace kvp {

// Philox counter tags: word 3 of the counter says what a block of random bits is for.
constexpr uint32_t TAG_MOVE = 1, TAG_CALIB = 2, TAG_NOISE = 3, TAG_BURST = 4, TAG_EXCHANGE = 6;   // 5: the (W, R) walk
constexpr uint32_t CALIB_N = 1024;

// Integer weights of Eq. 3-4, premultiplied with the migration flags.
struct CostK {
    uint32_t kh, ke;      // kappa_h, kappa_e
    uint32_t khF;         // kappa_h * Fh
    uint32_t kkF, kdF;    // kappa_k * Fe, kappa_d * Fe
    uint32_t kk, kd;      // kappa_k, kappa_d (writes are charged whatever the migration flags say)
};

// Per-step constants: x = kappa_h*hw, y = kappa_k*ew, z = kappa_d*ew, w = kappa_e*|A[s]|.
typedef uint4 StepC;

// Eq. 2-4 in ticks. All operands fit 31 bits (checked at kvp_create).
__device__ __forceinline__ uint32_t step_cost(uint32_t hr, uint32_t mi, uint32_t mo, const StepC c, const CostK k)
{
    const uint32_t mm = mi + mo;
    const uint32_t th = c.x + k.kh * hr + k.khF * mm;                 // Eq. 3
    const uint32_t e1 = c.y + k.kkF * mo;                             // link, towards DRAM
    const uint32_t e2 = k.kkF * mi;                                   // link, towards HBM
    const uint32_t e3 = c.z + k.kdF * mm;                             // DRAM channels
    const uint32_t te = c.w - k.ke * hr + max(max(e1, e2), e3);       // Eq. 4 (c.w - ke*hr = ke*|E^r|)
    return max(th, te);                                               // Eq. 2
}

// Philox4x32-10 (Salmon et al., SC'11).
__host__ __device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                        uint32_t k0, uint32_t k1, uint32_t out[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
#ifdef __CUDA_ARCH__
        const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
        const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
#else
        const uint64_t p0 = 0xD2511F53ull * c0, p1 = 0xCD9E8D57ull * c2;
        const uint32_t h0 = (uint32_t)(p0 >> 32), l0 = (uint32_t)p0, h1 = (uint32_t)(p1 >> 32), l1 = (uint32_t)p1;
#endif
        c0 = h1 ^ c1 ^ k0;
        c1 = l1;
        c2 = h0 ^ c3 ^ k1;
        c3 = l0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The ten round keys of Philox4x32-10 for one seed (round r uses key + r * Weyl constant). A kernel that draws every
// block with the same seed takes them as a launch parameter: the per-round additions then cost nothing on the device.
struct PhiloxKeys {
    uint32_t k0[10], k1[10];
};

inline PhiloxKeys philox_keys(uint32_t seed_lo, uint32_t seed_hi)
{
    PhiloxKeys k;
    for (int r = 0; r < 10; ++r) {
        k.k0[r] = seed_lo + (uint32_t)r * 0x9E3779B9u;
        k.k1[r] = seed_hi + (uint32_t)r * 0xBB67AE85u;
    }
    return k;
}

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, const PhiloxKeys& k,
                                              uint32_t out[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
        const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
        c0 = h1 ^ c1 ^ k.k0[r];
        c1 = l1;
        c2 = h0 ^ c3 ^ k.k1[r];
        c3 = l0;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The same with a growing cache: hb units are written to HBM at birth during this step. c.y and c.z count every
// unit born in the step as written to DRAM; each one that goes to HBM instead moves from |E^w| to |H^w|.
__device__ __forceinline__ uint32_t step_cost_g(uint32_t hr, uint32_t mi, uint32_t mo, uint32_t hb, const StepC c,
                                                const CostK k)
{
    const uint32_t mm = mi + mo;
    const uint32_t th = c.x + k.kh * (hr + hb) + k.khF * mm;          // Eq. 3
    const uint32_t e1 = c.y - k.kk * hb + k.kkF * mo;
    const uint32_t e2 = k.kkF * mi;
    const uint32_t e3 = c.z - k.kd * hb + k.kdF * mm;
    const uint32_t te = c.w - k.ke * hr + max(max(e1, e2), e3);       // Eq. 4
    return max(th, te);                                               // Eq. 2
}

}  // namespace kvp

// Host-side problem object behind the opaque handle.
struct kvp_problem {
    uint32_t U, S, W32, S32, cap;
    uint32_t pad_mask;          // valid bits of the last word of a step-major row
    uint32_t tail_mask;         // valid bits of the last word of a time-packed column
    uint64_t bytes_per_unit;
    uint64_t kh, kk, kd, ke, lcm, gcd;
    uint32_t mig_flags;
    double spt;
    int device;
    kvp::CostK K;
    uint32_t* dA;        // [S][W32]   access bitmap, step-major, pad bits clear
    uint32_t* dAcol;     // [U][S32]   access bitmap, time-packed (bit t of unit u = bit t&31 of word t>>5)
    uint32_t* d_a;       // [S]        |A[s]|
    kvp::StepC* d_stepc; // [S]
    uint32_t* d_ucnt;    // [U]        accesses per unit over all steps
    uint32_t* d_row_freq;// [W32]      STATIC_FREQ row
    uint64_t total_accessed;
    // growing cache (kvp_set_births); all null for a fixed population
    uint32_t* d_birth;   // [U]        step at which a unit is written, 0 = there from the start
    uint32_t* dL;        // [S][W32]   bit u of row s set iff unit u exists at step s
    void* d_grow_block;  // the allocation behind the two
    uint32_t* h_writes;  // (host) [S] hw + ew of kvp_create, for the range check of kvp_set_births
    void* d_block;             // one allocation behind the pointers above
    cudaStream_t last_stream;  // stream of the most recent call; frees are ordered behind it
    // scratch owned by the problem, grown on demand
    void* d_scratch; size_t scratch_bytes;
    void* d_chain_ws; size_t chain_ws_bytes;
};

namespace kvp {

int set_cuda_error(cudaError_t e, const char* what);
#define KVP_CUDA(call)                                                   \
    do {                                                                 \
        cudaError_t e_ = (call);                                         \
        if (e_ != cudaSuccess) return kvp::set_cuda_error(e_, #call);    \
    } while (0)

// keep freed blocks of up to `bytes` (+ 1 GiB) in the device's default memory pool
int retain_in_pool(int device, size_t bytes);
int ensure_scratch(kvp_problem* p, size_t bytes, cudaStream_t st);
int ensure_chain_ws(kvp_problem* p, size_t bytes, cudaStream_t st);

// kvp_cost.cu
int launch_row_popcount(const uint32_t* rows, uint32_t S, uint32_t W32, uint32_t* out, cudaStream_t st);
// hbc: [n][S] units written to HBM at birth; needed (and only used) when the problem has births
int launch_counts(const kvp_problem* p, const uint32_t* schedules, uint32_t n, uint32_t* counts, uint32_t* hbc,
                  cudaStream_t st, uint32_t* launches);
int launch_finish(const kvp_problem* p, const uint32_t* counts, const uint32_t* hbc, uint32_t n, uint64_t* step_ticks,
                  uint64_t* total_ticks, double* step_seconds, double* total_seconds, int32_t* bad_step, uint64_t* hits,
                  cudaStream_t st);

// kvp_layout.cu
int launch_bit_transpose(const uint32_t* in, uint32_t rows, uint32_t in_words, uint32_t cols, uint32_t* out,
                         uint32_t out_words, cudaStream_t st);
int launch_clean_copy(const uint32_t* in, uint32_t* out, uint32_t S, uint32_t W32, uint32_t pad_mask, cudaStream_t st);
int launch_unit_counts(const uint32_t* Acol, uint32_t U, uint32_t S32, uint32_t* ucnt, cudaStream_t st);
int launch_static_freq_row(const kvp_problem* p, uint32_t* row, cudaStream_t st);
int launch_static_first_row(const kvp_problem* p, uint32_t* row, cudaStream_t st);
int launch_broadcast_row(const uint32_t* row, uint32_t S, uint32_t W32, uint32_t* sched, cudaStream_t st);
int launch_row_to_columns(const uint32_t* row, uint32_t U, uint32_t S, uint32_t S32, uint32_t* Pcol, cudaStream_t st);
int launch_alive_rows(const uint32_t* birth, uint32_t U, uint32_t S, uint32_t W32, uint32_t* L, cudaStream_t st);
int launch_birth_stats(const uint32_t* birth, uint32_t U, uint32_t S, const uint32_t* Acol, uint32_t S32, uint32_t* nb,
                       uint32_t* flag, cudaStream_t st);
int launch_stepc_births(StepC* stepc, const uint32_t* nb, uint32_t S, uint32_t kk, uint32_t kd, cudaStream_t st);
int launch_and_rows(uint32_t* sched, const uint32_t* L, size_t total, cudaStream_t st);

}  // namespace kvp
