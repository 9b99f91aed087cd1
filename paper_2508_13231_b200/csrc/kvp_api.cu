// Host side of the C ABI: problem construction, integer time base, acceptance table, error text.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <thread>
#include <vector>

#include "kvp_common.cuh"

namespace kvp {

static thread_local char g_cuda_err[256] = "";

int set_cuda_error(cudaError_t e, const char* what)
{
    snprintf(g_cuda_err, sizeof g_cuda_err, "%s: %s", what, cudaGetErrorString(e));
    cudaGetLastError();  // clear the sticky-free error state
    return e == cudaErrorMemoryAllocation ? KVP_ERR_NOMEM : KVP_ERR_CUDA;
}

// All device memory comes from the stream-ordered allocator: a create/anneal/destroy cycle then costs no
// device-wide synchronisation. The default pool is told to keep freed memory up to the largest block this
// library has asked for on the device so far (at least 1 GiB), so that the next problem of the same size
// gets its workspace back without a trip to the driver.
int retain_in_pool(int device, size_t bytes)
{
    static uint64_t kept[64];                // racing threads may both raise the threshold; either value is fine
    if (device < 0 || device >= 64) return KVP_OK;
    uint64_t want = (uint64_t)bytes + (1ull << 30);
    if (__atomic_load_n(&kept[device], __ATOMIC_RELAXED) >= want) return KVP_OK;
    cudaMemPool_t pool;
    KVP_CUDA(cudaDeviceGetDefaultMemPool(&pool, device));
    uint64_t now = 0;
    KVP_CUDA(cudaMemPoolGetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &now));
    if (now < want) KVP_CUDA(cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &want));
    __atomic_store_n(&kept[device], want, __ATOMIC_RELAXED);
    return KVP_OK;
}

static int prepare_pool(int device) { return retain_in_pool(device, 0); }

static int grow(void** ptr, size_t* have, size_t want, cudaStream_t st)
{
    if (*have >= want) return KVP_OK;
    if (*ptr) { KVP_CUDA(cudaFreeAsync(*ptr, st)); *ptr = nullptr; *have = 0; }
    size_t bytes = (want + 255) & ~(size_t)255;
    int dev = 0;
    KVP_CUDA(cudaGetDevice(&dev));
    int rc = retain_in_pool(dev, bytes);
    if (rc) return rc;
    KVP_CUDA(cudaMallocAsync(ptr, bytes, st));
    *have = bytes;
    return KVP_OK;
}

int ensure_scratch(kvp_problem* p, size_t bytes, cudaStream_t st)
{
    p->last_stream = st;
    return grow(&p->d_scratch, &p->scratch_bytes, bytes, st);
}
int ensure_chain_ws(kvp_problem* p, size_t bytes, cudaStream_t st)
{
    p->last_stream = st;
    return grow(&p->d_chain_ws, &p->chain_ws_bytes, bytes, st);
}

static uint64_t gcd_u64(uint64_t a, uint64_t b)
{
    while (b) { const uint64_t t = a % b; a = b; b = t; }
    return a;
}

// kappa_x = L / (B_x / g): the smallest integers inversely proportional to the bandwidths of Eq. 3-4.
static int derive_weights(const kvp_memsys* m, kvp_problem* p)
{
    const uint64_t g = gcd_u64(gcd_u64(m->bw_hbm, m->bw_link), m->bw_dram);
    const uint64_t rh = m->bw_hbm / g, rk = m->bw_link / g, rd = m->bw_dram / g;
    const uint64_t limit = 1ull << 40;
    uint64_t L = rh / gcd_u64(rh, rk);
    if (L > limit / rk) return KVP_ERR_RANGE;
    L *= rk;
    const uint64_t Lq = L / gcd_u64(L, rd);
    if (Lq > limit / rd) return KVP_ERR_RANGE;
    L = Lq * rd;
    p->gcd = g; p->lcm = L;
    p->kh = L / rh; p->kk = L / rk; p->kd = L / rd;
    p->ke = p->kk > p->kd ? p->kk : p->kd;
    return KVP_OK;
}

}  // namespace kvp

using namespace kvp;

extern "C" void kvp_destroy(kvp_problem* p)
{
    if (!p) return;
    cudaSetDevice(p->device);
    // freed in stream order behind the last work queued for this problem
    if (p->d_block) cudaFreeAsync(p->d_block, p->last_stream);
    if (p->d_scratch) cudaFreeAsync(p->d_scratch, p->last_stream);
    if (p->d_chain_ws) cudaFreeAsync(p->d_chain_ws, p->last_stream);
    if (p->d_grow_block) cudaFreeAsync(p->d_grow_block, p->last_stream);
    free(p->h_writes);
    delete p;
}

static int create_impl(kvp_problem* p, const uint32_t* access, const uint32_t* hw, const uint32_t* ew, cudaStream_t st)
{
    const size_t nw = (size_t)p->S * p->W32;
    int rc = prepare_pool(p->device);
    if (rc) return rc;
    p->last_stream = st;
    // one block for everything the problem keeps
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 255) & ~(size_t)255; return o; };
    const size_t oA = take(nw * 4), oAcol = take((size_t)p->U * p->S32 * 4), oa = take((size_t)p->S * 4);
    const size_t osc = take((size_t)p->S * sizeof(StepC)), ouc = take((size_t)p->U * 4), orf = take((size_t)p->W32 * 4);
    KVP_CUDA(cudaMallocAsync(&p->d_block, off, st));
    char* base = static_cast<char*>(p->d_block);
    p->dA = (uint32_t*)(base + oA); p->dAcol = (uint32_t*)(base + oAcol); p->d_a = (uint32_t*)(base + oa);
    p->d_stepc = (StepC*)(base + osc); p->d_ucnt = (uint32_t*)(base + ouc); p->d_row_freq = (uint32_t*)(base + orf);
    // what launch_static_freq_row needs: histogram, selection, tie counts of the chunks of 1024 units
    if ((rc = ensure_scratch(p, (size_t)(p->S + 8) * 16 + ((size_t)p->W32 / 32 + 2) * 4, st))) return rc;
    if ((rc = launch_clean_copy(access, p->dA, p->S, p->W32, p->pad_mask, st))) return rc;
    if ((rc = launch_row_popcount(p->dA, p->S, p->W32, p->d_a, st))) return rc;
    if ((rc = launch_bit_transpose(p->dA, p->S, p->W32, p->U, p->dAcol, p->S32, st))) return rc;
    if ((rc = launch_unit_counts(p->dAcol, p->U, p->S32, p->d_ucnt, st))) return rc;
    if ((rc = launch_static_freq_row(p, p->d_row_freq, st))) return rc;
    std::vector<uint32_t> a(p->S);
    KVP_CUDA(cudaMemcpyAsync(a.data(), p->d_a, (size_t)p->S * 4, cudaMemcpyDeviceToHost, st));
    KVP_CUDA(cudaStreamSynchronize(st));
    // Per-step constants of the cost function; everything must stay below 2^31 so that the
    // annealer can work in 32-bit arithmetic.
    uint64_t wmax = 0;
    p->h_writes = static_cast<uint32_t*>(malloc((size_t)p->S * 4));
    if (!p->h_writes) return KVP_ERR_NOMEM;
    for (uint32_t s = 0; s < p->S; ++s) {
        const uint64_t e = (uint64_t)(hw ? hw[s] : 0) + (ew ? ew[s] : 0);
        if (e >= (1ull << 31)) return KVP_ERR_RANGE;
        p->h_writes[s] = (uint32_t)e;
        if (e > wmax) wmax = e;
    }
    const uint64_t kmax = p->kh > p->ke ? p->kh : p->ke;
    if (kmax * (2ull * p->U + wmax) >= (1ull << 31)) return KVP_ERR_RANGE;
    std::vector<StepC> sc(p->S);
    p->total_accessed = 0;
    for (uint32_t s = 0; s < p->S; ++s) {
        const uint64_t h = hw ? hw[s] : 0, e = ew ? ew[s] : 0;
        sc[s] = make_uint4((uint32_t)(p->kh * h), (uint32_t)(p->kk * e), (uint32_t)(p->kd * e), (uint32_t)(p->ke * a[s]));
        p->total_accessed += a[s];
    }
    KVP_CUDA(cudaMemcpyAsync(p->d_stepc, sc.data(), (size_t)p->S * sizeof(StepC), cudaMemcpyHostToDevice, st));
    KVP_CUDA(cudaStreamSynchronize(st));
    return KVP_OK;
}

extern "C" int kvp_create(kvp_problem** out, uint32_t units, uint64_t bytes_per_unit, uint32_t steps,
                          const uint32_t* access_bitmaps, uint32_t hbm_capacity_units, const kvp_memsys* mem,
                          const uint32_t* hw_units, const uint32_t* ew_units, void* stream)
{
    if (!out || !access_bitmaps || !mem || !units || !steps || !bytes_per_unit) return KVP_ERR_ARG;
    if (hbm_capacity_units > units || mem->reserved || (mem->mig_flags & ~KVP_MIG_PAPER)) return KVP_ERR_ARG;
    if (!mem->bw_hbm || !mem->bw_link || !mem->bw_dram) return KVP_ERR_ARG;
    if (units >= (1u << 26) || steps > 32768) return KVP_ERR_RANGE;
    int dev = 0;
    KVP_CUDA(cudaGetDevice(&dev));
    kvp_problem* p = new (std::nothrow) kvp_problem();
    if (!p) return KVP_ERR_NOMEM;
    memset(p, 0, sizeof *p);
    p->device = dev;
    p->U = units; p->S = steps; p->cap = hbm_capacity_units;
    p->W32 = (units + 31) / 32; p->S32 = (steps + 31) / 32;
    p->pad_mask = units % 32 ? (1u << (units % 32)) - 1u : 0xFFFFFFFFu;
    p->tail_mask = steps % 32 ? (1u << (steps % 32)) - 1u : 0xFFFFFFFFu;
    p->bytes_per_unit = bytes_per_unit;
    p->mig_flags = mem->mig_flags;
    int rc = derive_weights(mem, p);
    if (rc) { delete p; return rc; }
    p->spt = (double)bytes_per_unit / ((double)p->lcm * (double)p->gcd);
    const uint32_t Fh = (mem->mig_flags & KVP_MIG_HBM) ? 1u : 0u, Fe = (mem->mig_flags & KVP_MIG_EXT) ? 1u : 0u;
    if (p->kh >= (1ull << 31) || p->ke >= (1ull << 31)) { delete p; return KVP_ERR_RANGE; }
    p->K.kh = (uint32_t)p->kh; p->K.ke = (uint32_t)p->ke;
    p->K.khF = (uint32_t)p->kh * Fh; p->K.kkF = (uint32_t)p->kk * Fe; p->K.kdF = (uint32_t)p->kd * Fe;
    p->K.kk = (uint32_t)p->kk; p->K.kd = (uint32_t)p->kd;
    rc = create_impl(p, access_bitmaps, hw_units, ew_units, static_cast<cudaStream_t>(stream));
    if (rc) { kvp_destroy(p); return rc; }
    *out = p;
    return KVP_OK;
}

extern "C" int kvp_set_births(kvp_problem* p, const uint32_t* birth, void* stream)
{
    if (!p || !birth || p->dL) return KVP_ERR_ARG;
    KVP_CUDA(cudaSetDevice(p->device));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p->last_stream = st;
    const size_t nw = (size_t)p->S * p->W32;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 255) & ~(size_t)255; return o; };
    const size_t ob = take((size_t)p->U * 4), oL = take(nw * 4), onb = take((size_t)p->S * 4 + 4);
    void* block = nullptr;
    KVP_CUDA(cudaMallocAsync(&block, off, st));
    char* base = static_cast<char*>(block);
    uint32_t* d_birth = (uint32_t*)(base + ob);
    uint32_t* dL = (uint32_t*)(base + oL);
    uint32_t* d_nb = (uint32_t*)(base + onb);            // [S] births per step, then the check flags
    std::vector<uint32_t> nb((size_t)p->S + 1);
    int rc = KVP_OK;
    auto fail = [&](int code) { cudaFreeAsync(block, st); return code; };
    if (cudaMemcpyAsync(d_birth, birth, (size_t)p->U * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
        cudaMemsetAsync(d_nb, 0, (size_t)p->S * 4 + 4, st) != cudaSuccess)
        return fail(set_cuda_error(cudaGetLastError(), "kvp_set_births copy"));
    if ((rc = launch_birth_stats(d_birth, p->U, p->S, p->dAcol, p->S32, d_nb, d_nb + p->S, st))) return fail(rc);
    if ((rc = launch_alive_rows(d_birth, p->U, p->S, p->W32, dL, st))) return fail(rc);
    if (cudaMemcpyAsync(nb.data(), d_nb, (size_t)p->S * 4 + 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return fail(set_cuda_error(cudaGetLastError(), "kvp_set_births read-back"));
    if (nb[p->S]) return fail(KVP_ERR_ARG);              // a birth beyond the horizon, or an access before birth
    uint64_t wmax = 0;
    for (uint32_t s = 0; s < p->S; ++s) {
        const uint64_t e = (uint64_t)p->h_writes[s] + nb[s];
        if (e > wmax) wmax = e;
    }
    const uint64_t kmax = p->kh > p->ke ? p->kh : p->ke;
    if (kmax * (2ull * p->U + wmax) >= (1ull << 31)) return fail(KVP_ERR_RANGE);
    if ((rc = launch_stepc_births(p->d_stepc, d_nb, p->S, p->K.kk, p->K.kd, st))) return fail(rc);
    p->d_grow_block = block; p->d_birth = d_birth; p->dL = dL;
    return KVP_OK;
}

extern "C" int kvp_get_info(const kvp_problem* p, kvp_info* info)
{
    if (!p || !info) return KVP_ERR_ARG;
    info->kappa_h = p->kh; info->kappa_k = p->kk; info->kappa_d = p->kd; info->kappa_e = p->ke;
    info->lcm = p->lcm; info->gcd = p->gcd; info->seconds_per_tick = p->spt;
    info->units = p->U; info->steps = p->S; info->words_per_row = p->W32; info->capacity = p->cap;
    return KVP_OK;
}

namespace {

// The rows rows[i0..i1) of the acceptance table. Entries whose exponent is beyond 22.5 > ln(2^32) are zero whatever
// the last bits of exp() are, so exp() is not called for them.
void accept_rows(const double* temps, const uint32_t* shifts, const uint32_t* rows, uint32_t i0, uint32_t i1,
                 uint32_t* table)
{
    for (uint32_t i = i0; i < i1; ++i) {
        const uint32_t j = rows[i];
        const double C = temps[j] >= 1.0 ? temps[j] : 1.0;     // also maps NaN to 1
        const double bin = (double)(1ull << shifts[j]);
        for (uint32_t q = 0; q < KVP_TABLE_Q; ++q) {
            const double x = ((double)q + 0.5) * bin;
            const double y = x / C;
            uint32_t v = 0u;
            if (y <= 22.5) {
                const double thr = 4294967296.0 * exp(-x / C);
                v = thr >= 4294967295.0 ? 0xFFFFFFFFu : (uint32_t)thr;
            }
            table[(size_t)j * KVP_TABLE_Q + q] = v;
        }
    }
}

}  // namespace

extern "C" int kvp_accept_table(const double* temps, uint32_t levels, uint32_t* table, uint32_t* shifts)
{
    if (!temps || !table || !shifts || !levels) return KVP_ERR_ARG;
    // A level whose (clamped) temperature equals that of the level before it has the same row: a ladder that has
    // cooled below one tick repeats its last row, often for a third of its levels. Only the others are computed.
    std::vector<uint32_t> rows;
    rows.reserve(levels);
    double prev = 0.0;
    for (uint32_t j = 0; j < levels; ++j) {
        const double C = temps[j] >= 1.0 ? temps[j] : 1.0;
        uint32_t sh = 0;
        while ((double)KVP_TABLE_Q * (double)(1ull << sh) < 23.0 * C)
            if (++sh > 40) return KVP_ERR_RANGE;
        shifts[j] = sh;
        if (j == 0 || C != prev) rows.push_back(j);
        prev = C;
    }
    const uint32_t nrows = (uint32_t)rows.size();
    // A ladder of 64 levels is up to 65,536 calls of exp(), about half a millisecond on one core and a tenth of an
    // annealing call on a small problem: the rows are independent, so a few threads share them.
    uint32_t nthr = nrows >= 16 ? std::min<uint32_t>(8u, std::max(1u, std::thread::hardware_concurrency())) : 1u;
    if (nthr > 1) {
        std::vector<std::thread> pool;
        const uint32_t per = (nrows + nthr - 1) / nthr;
        try {
            for (uint32_t t = 1; t < nthr && t * per < nrows; ++t)
                pool.emplace_back(accept_rows, temps, shifts, rows.data(), t * per, std::min(nrows, (t + 1) * per), table);
        } catch (...) {                                        // no thread to be had: this one does the rest
            const uint32_t done = (uint32_t)pool.size() + 1;
            accept_rows(temps, shifts, rows.data(), std::min(nrows, done * per), nrows, table);
        }
        accept_rows(temps, shifts, rows.data(), 0, std::min(nrows, per), table);
        for (auto& th : pool) th.join();
    } else {
        accept_rows(temps, shifts, rows.data(), 0, nrows, table);
    }
    for (uint32_t j = 1, i = 1; j < levels; ++j) {             // the repeated rows, each from the row before it
        if (i < nrows && rows[i] == j) { ++i; continue; }
        memcpy(table + (size_t)j * KVP_TABLE_Q, table + (size_t)(j - 1) * KVP_TABLE_Q, KVP_TABLE_Q * sizeof(uint32_t));
    }
    return KVP_OK;
}

extern "C" void kvp_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    philox4x32_10(ctr[0], ctr[1], ctr[2], ctr[3], key[0], key[1], out);
}

extern "C" const char* kvp_strerror(int code)
{
    switch (code) {
        case KVP_OK: return "ok";
        case KVP_ERR_ARG: return "invalid argument";
        case KVP_ERR_CAPACITY: return "schedule exceeds the HBM capacity (Eq. 5)";
        case KVP_ERR_RANGE: return "size or weight outside the supported integer range";
        case KVP_ERR_CUDA: return "CUDA runtime error";
        case KVP_ERR_NOMEM: return "out of memory";
        case KVP_ERR_TIMEOUT: return "device-side wait timed out";
        case KVP_ERR_INTERNAL: return "internal self-check failed";
        default: return "unknown error";
    }
}

extern "C" const char* kvp_last_cuda_error(void) { return kvp::g_cuda_err; }
