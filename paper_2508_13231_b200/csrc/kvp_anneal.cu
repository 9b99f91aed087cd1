// Annealing kernels. Two of them, chosen per job (see prepare()): the narrow chain kernel described here (one or two
// warps per chain, one proposal per lane) and the wide one further down (one warp per chain, four proposals per lane,
// most proposals settled by their placement bits alone).
//
// State of a chain: the schedule in time-packed form (for every unit a bit string over the steps), either
// in shared memory (small problems) or in a private slice of global scratch (a plain copy of the initial schedule,
// or a copy-on-write overlay of the one all chains share), plus the four per-step cardinalities {hr, mi, mo, occ}
// in shared memory and the running total T.
//
// A proposal (one Philox4x32-10 block, a pure function of seed, chain and move index) names a run of at most
// 30 consecutive steps and one or two units. Only the run's steps and the step after it change cost. Proposals
// are drawn and evaluated 32 at a time, one per lane, against the state the batch starts from; the (proposal,
// step) pairs whose cost changes go through a work queue shared by the warp; the warp then commits the batch in
// move order with a Metropolis test against the quantised exp(-delta/C) table, evaluating again only what an
// applied move could have touched. With two warps per chain the warps take the batches in turn (see ChainShare).
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <type_traits>
#include <vector>

#include "kvp_common.cuh"

namespace kvp {

namespace {

kvp_test_hooks g_hooks = {0u, 0u, 0u, 0u, 0u};   // kvp_set_test_hooks; read once per call

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
    const uint32_t* full0;       // [S32] full-step bitmap of the initial schedule
    uint32_t* snap;              // if set: [slots][U*S32], each chain's schedule when it reached its best
    uint64_t* undo_log;          // if set: [slots][undo_cap] indices of the moves applied since the best state
    uint32_t* undo_len;          // [slots] how many there were (more than undo_cap: the log overflowed)
    uint32_t undo_cap;
    uint32_t* err;               // set to 1 by a warp that gave up waiting for its turn
    uint32_t drop_first_turn;    // test hook: the owner of batch 0 never passes the turn on, so the next wait runs out
    uint32_t split_at;           // a batch with more queue items than this goes in two halves (kQueueCap / 2; less in tests)
    const uint32_t* birth;       // growing cache: [U] step at which a unit is written (0 = there from the start)
    const uint32_t* hb0;         // growing cache: [S] units written to HBM at birth under the initial schedule
    CostK K;
    uint32_t U, S, S32, cap;
    uint32_t chain_first, chain_count, result_base;
    uint32_t levels, p_swap_256, len_choices;
    uint32_t early_permille, early_from;
    PhiloxKeys keys;             // round keys of the seed
    uint64_t per_level, upto, init_ticks;
    uint32_t* cow_out;           // wide kernel, schedules in global scratch: [slots][cow_slots4 * 4] which buckets of
                                 // units a slot's slice holds when its chain ends (the rest is the initial schedule)
    uint32_t cow_shift;          // a bucket is 2^cow_shift consecutive units
    uint32_t stage_stepc;        // wide kernel without a staged access bitmap: the step constants alone are staged
    unsigned long long* work;    // wide kernel: [3] sums over the chains of {n_again, n_listed, n_items}
    // Replica exchange (wide kernel): the call runs rounds round0 .. round1-1; in round t chain c proposes moves
    // t * exch_every .. (t + 1) * exch_every - 1 (up to `upto`) with the table row of the rung it holds,
    // rung_hist[t * hist_stride + (c - hist_base)].
    const uint8_t* rung_hist;    // null: the ordinary cooling schedule by temperature levels
    uint64_t exch_every;
    uint32_t round0, round1, hist_stride, hist_base;
    uint4* state;                // if set: [chains][state4] the chain's persistent shared-memory state (and its
                                 // schedule, when that lives in shared memory), indexed like rung_hist
    uint32_t state4;             // uint4 slots per chain in `state`
    uint32_t resume;             // 1: start from `state` instead of the initial schedule
    uint32_t cow_slots4;         // schedules in global scratch: uint4 slots of a chain's bucket bitmap; 0 (narrow kernel
                                 // only): plain slices, each a whole copy of the initial schedule
};

// Batches: every lane of a chain's warp carries kMPL proposals, so a batch is 32 * kMPL consecutive moves.
// Measured on 256 units x 512 steps, 1024 chains: kMPL = 2 is slower (6.0 ms vs 5.25 ms per 10^8 moves): a move that
// changes the schedule then costs a re-evaluation pass over twice as many proposals. Serving a chain with two warps
// that evaluate side by side and commit in turn was tried as well and was no faster (5.9 ms).
constexpr int kMPL = 1;
constexpr uint32_t kBatch = 32 * kMPL;
constexpr uint32_t kWinSlots4 = kBatch * 2;                        // 8 words of windows per proposal
constexpr uint32_t kAccSlots4 = kBatch / 4;                        // one int per proposal
// uint16 work items, 31 per proposal in the worst case. Where shared memory is short (HALFQ) the queue holds the worst
// case of half a warp's proposals and a batch with more items than that is worked off in two halves.
constexpr uint32_t kQueueCap = kBatch * 31;
constexpr uint32_t kQueueSlots4 = (kQueueCap * 2 + 15) / 16;
constexpr uint32_t kHalfQueueSlots4 = (kQueueCap / 2 * 2 + 15) / 16;

// A proposal as its lane keeps it in registers: the Philox words and, after evaluation, the verdict.
// The placement windows live in shared memory (ChainView::win), 8 words per proposal:
//   {Wu, Wv, Nu, Nv} = placement of units u, v before (W) and after (N) the move, {Au, Av} = access bits,
//   then s0. Window convention: bit k belongs to step s0 - 1 + k, so bit 0 is the step before the run (for
//   s0 == 0 it repeats step 0, because P[-1] := P[0]), bits 1..run are the run, and the affected steps
//   s0..last are bits 1..nl <= 31. Run lengths stop at 30 so that every vector fits one 32-bit register.
struct LaneMove {
    uint32_t pk, u, v, w;        // packed (swap | len << 1 | s0 << 8), units, Metropolis uniform
    int delta;
    bool inf, acc, chg;
};

__device__ __forceinline__ void decode_move(const uint32_t r[4], uint32_t p_swap_256, uint32_t len_choices, uint32_t S,
                                            uint32_t U, LaneMove& mv)
{
    const uint32_t swap = (r[0] & 255u) < p_swap_256 ? 1u : 0u;
    const uint32_t k = (((r[0] >> 8) & 255u) * len_choices) >> 8;
    const uint32_t len = min(1u << k, 30u);
    const uint32_t s0 = ((r[0] >> 16) * S) >> 16;
    mv.pk = swap | (len << 1) | (s0 << 8);
    mv.u = __umulhi(r[1], U);
    mv.v = __umulhi(r[2], U);
    mv.w = r[3];
}

// 32 consecutive bits of a time-packed column starting at step s0 - 1 (see LaneMove). Bits that belong to
// steps beyond the horizon are arbitrary; every user masks them.
template <typename Ptr>
__device__ __forceinline__ uint32_t window(Ptr col, uint32_t S32, uint32_t s0)
{
    const uint32_t b0 = s0 ? s0 - 1 : 0u, w = b0 >> 5;
    const uint32_t lo = col[w], hi = col[min(w + 1, S32 - 1)];
    const uint32_t slid = __funnelshift_r(lo, hi, b0 & 31u);
    return s0 ? slid : ((lo << 1) | (lo & 1u));                  // s0 == 0: bit 0 repeats step 0
}

// The same cut for several columns of one proposal: the position is worked out once.
struct WinPos {
    uint32_t w, w2, sh;          // first word, the word after it (clamped), shift
    bool first;                  // s0 == 0: bit 0 repeats step 0
};
__device__ __forceinline__ WinPos window_pos(uint32_t S32, uint32_t s0)
{
    WinPos p;
    const uint32_t b0 = s0 ? s0 - 1 : 0u;
    p.w = b0 >> 5; p.w2 = min(p.w + 1, S32 - 1); p.sh = b0 & 31u; p.first = s0 == 0;
    return p;
}
// COLV = 2 or 4: every column is exactly that many words (at most 64 or 128 steps) and comes with one vector load: a
// warp's 32 columns are 32 different lines, and what limits the chains in global memory is the number of such
// scattered loads. (Every column then starts on an 8- or 16-byte boundary; the arrays themselves are 16-byte
// aligned.) COLV = 0: columns of any length, the two words they need. The choice is made at compile time: a test of
// S32 around every load breaks up the straight-line block in which all loads of a batch are issued, and was 1.5x slower.
template <int COLV, typename Ptr>
__device__ __forceinline__ uint32_t window_at(Ptr col, const WinPos p)
{
    uint32_t lo, hi;
    if (COLV == 2) {
        const uint2 q = *reinterpret_cast<const uint2*>(col);
        lo = p.w ? q.y : q.x;
        hi = q.y;
    } else if (COLV == 4) {
        const uint4 q = *reinterpret_cast<const uint4*>(col);
        lo = p.w == 0 ? q.x : p.w == 1 ? q.y : p.w == 2 ? q.z : q.w;
        hi = p.w == 0 ? q.y : p.w == 1 ? q.z : q.w;
    } else {
        lo = col[p.w];
        hi = col[p.w2];
    }
    return p.first ? ((lo << 1) | (lo & 1u)) : __funnelshift_r(lo, hi, p.sh);
}

struct ChainView {               // where a chain's state lives
    uint32_t* P;                 // [U][S32] schedule, time-packed (shared, or the chain's slice of global scratch)
    // COW (a compile-time choice of the kernel): the slice of global scratch is a copy-on-write overlay of the initial
    // schedule p0 (see kCowBitsMin) and `have` says which buckets of 2^shift units it holds. Otherwise the schedule is
    // all in P.
    const uint32_t* p0;
    uint32_t* have;
    uint32_t shift, U, S32;
    bool shared_chain;           // a second warp of the chain reads while this one commits
    template <bool COW>
    __device__ __forceinline__ const uint32_t* col(uint32_t u) const
    {
        if (COW) {
            const uint32_t b = u >> shift;
            // volatile: another warp of the chain may be taking the bucket over meanwhile (it sets the bit after the
            // copy); a select, not a branch, so that the loads of a batch stay in one straight-line block
            const uint32_t w = reinterpret_cast<const volatile uint32_t*>(have)[b >> 5];
            return ((w >> (b & 31u)) & 1u ? P : p0) + (size_t)u * S32;
        }
        return P + (size_t)u * S32;
    }
    // Before unit u is rewritten (all lanes of the committing warp, u uniform): its bucket is copied into the slice.
    template <bool COW>
    __device__ __forceinline__ void own(uint32_t u, uint32_t lane) const
    {
        if (!COW) return;
        const uint32_t b = u >> shift;
        if ((have[b >> 5] >> (b & 31u)) & 1u) return;
        const size_t lo = (size_t)(b << shift) * S32, hi = (size_t)min(U, (b + 1u) << shift) * S32;
        for (size_t i = lo + lane; i < hi; i += 32) P[i] = p0[i];
        if (shared_chain) __threadfence_block();                  // the copy before the bit, for the chain's other warp
        __syncwarp();
        if (lane == 0) have[b >> 5] |= 1u << (b & 31u);
        __syncwarp();
    }
    uint4* ctr;                  // [S] {hr, mi, mo, occ} (shared)
    uint32_t* full;              // [S32] bit t set iff occ[t] == cap (shared)
    uint4* win;                  // [kBatch][2] windows of the batch's proposals (shared)
    int* acc;                    // [kBatch] cost change of each proposal being summed (shared)
    uint16_t* queue;             // [kBatch * 31] work items (proposal slot << 5 | window bit) (shared)
    uint32_t* hb;                // growing cache: [S] units written to HBM at birth (shared)
};

// born: window bit of the step in which u (low byte) and v (next byte) are written, 0 = not among bits 1..31
struct Windows { uint32_t Wu, Wv, Nu, Nv, Au, Av, s0, born; };

// Growing cache, unit with birth step b seen through the window that starts at step s0 - 1 (-1 for s0 == 0):
// the bits of steps at which it exists, and the bit of the step in which it is written.
__device__ __forceinline__ void alive_born(uint32_t b, uint32_t s0, uint32_t& alive, uint32_t& born)
{
    const int off = (int)b - ((int)s0 - 1);
    alive = (b == 0 || off <= 0) ? 0xFFFFFFFFu : (off >= 32 ? 0u : 0xFFFFFFFFu << off);
    born = (b != 0 && off >= 1 && off < 32) ? 1u << off : 0u;
}

// First half of evaluating a proposal, all in the calling lane and word-parallel over the <= 31 affected
// steps: the windows before and after the move, feasibility (Eq. 5), whether any bit changes, and the set
// of window bits (steps) whose cardinalities, hence cost, change.
// GROW: a move acts only on the steps at which the units it names exist, and a unit that enters HBM in the step
// it is written was written there (it counts in hb), not migrated.
// colu, colv: the time-packed placement columns of unit u and of unit v (of u again for a flip).
template <bool GROW, typename PPtr, typename FPtr>
__device__ __forceinline__ uint32_t lane_windows(PPtr colu, PPtr colv, const uint32_t* __restrict__ Acol, FPtr full,
                                                 const uint32_t* __restrict__ birth, uint32_t S, uint32_t S32,
                                                 LaneMove& mv, Windows& wn)
{
    const bool swap = mv.pk & 1u;
    const uint32_t len = (mv.pk >> 1) & 63u, s0 = mv.pk >> 8;
    const uint32_t run = min(s0 + len, S) - s0;                   // steps whose placement bits change hands
    const uint32_t nl = min(s0 + len, S - 1) - s0 + 1;            // affected steps: the run and the step after it
    const uint32_t M = ((1u << run) - 1u) << 1;
    const uint32_t Sb = ((1u << nl) - 1u) << 1;
    // branch-free: a flip reads unit u twice and ignores the second copy, a swap ignores the full-step window
    const size_t ub = (size_t)mv.u * S32, vb = (size_t)(swap ? mv.v : mv.u) * S32;
    const uint32_t Wu = window(colu, S32, s0), Au = window(Acol + ub, S32, s0);
    const uint32_t wv = window(colv, S32, s0), av = window(Acol + vb, S32, s0);
    const uint32_t Wv = swap ? wv : 0u, Av = swap ? av : 0u;
    const uint32_t Fw = window(full, S32, s0);
    uint32_t Bu = 0u, Bv = 0u, live = 0xFFFFFFFFu;
    if (GROW) {
        uint32_t Lu, Lv;
        alive_born(__ldg(birth + mv.u), s0, Lu, Bu);
        alive_born(__ldg(birth + (swap ? mv.v : mv.u)), s0, Lv, Bv);
        live = Lu & Lv;
        if (!swap) Bv = 0u;
    }
    const uint32_t D = (swap ? (Wu ^ Wv) : 0xFFFFFFFFu) & M & live;      // bits that toggle
    uint32_t Nu = Wu ^ D, Nv = swap ? (Wv ^ D) : 0u;
    if (s0 == 0) {                                                // the virtual step -1 follows step 0
        Nu = (Nu & ~1u) | ((Nu >> 1) & 1u);
        Nv = (Nv & ~1u) | ((Nv >> 1) & 1u);
    }
    wn.Wu = Wu; wn.Wv = Wv; wn.Nu = Nu; wn.Nv = Nv; wn.Au = Au; wn.Av = Av; wn.s0 = s0;
    wn.born = GROW ? ((Bu ? 31u - __clz(Bu) : 0u) | ((Bv ? 31u - __clz(Bv) : 0u) << 8)) : 0u;
    mv.chg = D != 0;
    mv.inf = !swap && (~Wu & D & Fw) != 0;                        // a flip may not raise a full step (Eq. 5)
    const uint32_t hr = (Au ^ Av) & (Wu ^ Nu);                    // a hit is won or lost (v mirrors u in a swap)
    // migrations of a unit at step t are the edges p[t] != p[t-1] (into HBM when p[t] is set, out otherwise):
    // the counts change where an edge appears, disappears or turns around
    // (the edge into the step of birth is no migration; there the placement bit moves a write between H^w and E^w)
    const uint32_t euo = (Wu ^ (Wu << 1)) & ~Bu, eun = (Nu ^ (Nu << 1)) & ~Bu;
    const uint32_t evo = (Wv ^ (Wv << 1)) & ~Bv, evn = (Nv ^ (Nv << 1)) & ~Bv;
    const uint32_t mg = (euo ^ eun) | (euo & eun & (Wu ^ Nu)) | (evo ^ evn) | (evo & evn & (Wv ^ Nv));
    const uint32_t wr = ((Wu ^ Nu) & Bu) | ((Wv ^ Nv) & Bv);
    return mv.inf ? 0u : ((hr | mg | wr) & Sb);
}

// Cost change of the step at window bit k (Eq. 2-4 before and after), from the windows of a proposal.
// hb: the step's count of units written to HBM at birth (GROW only).
template <bool GROW>
__device__ __forceinline__ int item_delta(const Windows& wn, uint32_t k, const uint4 c4, uint32_t hb, const StepC c,
                                          const CostK K)
{
    const uint32_t pu = (wn.Wu >> k) & 1u, qu = (wn.Wu >> (k - 1)) & 1u, npu = (wn.Nu >> k) & 1u, nqu = (wn.Nu >> (k - 1)) & 1u;
    const uint32_t pv = (wn.Wv >> k) & 1u, qv = (wn.Wv >> (k - 1)) & 1u, npv = (wn.Nv >> k) & 1u, nqv = (wn.Nv >> (k - 1)) & 1u;
    const uint32_t au = (wn.Au >> k) & 1u, av = (wn.Av >> k) & 1u;
    const uint32_t hr = c4.x + (au & npu) - (au & pu) + (av & npv) - (av & pv);
    if (GROW) {
        // mu / mv: 1 when the step is an ordinary one for the unit, 0 when it is the step the unit is written in
        const uint32_t mu = (wn.born & 255u) == k ? 0u : 1u, mw = ((wn.born >> 8) & 255u) == k ? 0u : 1u;
        const uint32_t mi = c4.y + mu * ((npu & ~nqu) - (pu & ~qu)) + mw * ((npv & ~nqv) - (pv & ~qv));
        const uint32_t mo = c4.z + (~npu & nqu & 1u) - (~pu & qu & 1u) + (~npv & nqv & 1u) - (~pv & qv & 1u);
        const uint32_t hn = hb + (1u - mu) * (npu - pu) + (1u - mw) * (npv - pv);
        return (int)(step_cost_g(hr, mi, mo, hn, c, K) - step_cost_g(c4.x, c4.y, c4.z, hb, c, K));
    }
    const uint32_t mi = c4.y + (npu & ~nqu) - (pu & ~qu) + (npv & ~nqv) - (pv & ~qv);
    const uint32_t mo = c4.z + (~npu & nqu & 1u) - (~pu & qu & 1u) + (~npv & nqv & 1u) - (~pv & qv & 1u);
    return (int)(step_cost(hr, mi, mo, c, K) - step_cost(c4.x, c4.y, c4.z, c, K));
}

// Cost of the step at window bit k after the proposal (Eq. 2-4), from its windows and the step's present counters.
template <bool GROW>
__device__ __forceinline__ uint32_t item_cost_after(const Windows& wn, uint32_t k, const uint4 c4, uint32_t hb, const StepC c,
                                                    const CostK K)
{
    const uint32_t pu = (wn.Wu >> k) & 1u, qu = (wn.Wu >> (k - 1)) & 1u, npu = (wn.Nu >> k) & 1u, nqu = (wn.Nu >> (k - 1)) & 1u;
    const uint32_t pv = (wn.Wv >> k) & 1u, qv = (wn.Wv >> (k - 1)) & 1u, npv = (wn.Nv >> k) & 1u, nqv = (wn.Nv >> (k - 1)) & 1u;
    const uint32_t au = (wn.Au >> k) & 1u, av = (wn.Av >> k) & 1u;
    const uint32_t hr = c4.x + (au & npu) - (au & pu) + (av & npv) - (av & pv);
    const uint32_t mo = c4.z + (~npu & nqu & 1u) - (~pu & qu & 1u) + (~npv & nqv & 1u) - (~pv & qv & 1u);
    if (GROW) {
        const uint32_t mu = (wn.born & 255u) == k ? 0u : 1u, mw = ((wn.born >> 8) & 255u) == k ? 0u : 1u;
        const uint32_t mi = c4.y + mu * ((npu & ~nqu) - (pu & ~qu)) + mw * ((npv & ~nqv) - (pv & ~qv));
        const uint32_t hn = hb + (1u - mu) * (npu - pu) + (1u - mw) * (npv - pv);
        return step_cost_g(hr, mi, mo, hn, c, K);
    }
    const uint32_t mi = c4.y + (npu & ~nqu) - (pu & ~qu) + (npv & ~nqv) - (pv & ~qv);
    return step_cost(hr, mi, mo, c, K);
}

__device__ __forceinline__ bool metropolis(int delta, uint32_t w, const uint32_t* __restrict__ trow, uint32_t shift)
{
    // branch-free: the threshold is loaded whatever delta is (a clamped index), so that the loads of several
    // proposals are in flight together instead of each behind its own branch
    const uint32_t q = (uint32_t)max(delta, 0) >> shift;
    const uint32_t thr = __ldg(trow + min(q, (uint32_t)KVP_TABLE_Q - 1u));
    return delta <= 0 || (q < KVP_TABLE_Q && w < thr);            // quantised exp(-delta/C)
}

// Whole evaluation in one lane (used where there is no warp to share the work with: calibration).
template <bool GROW, typename PPtr, typename CPtr, typename FPtr>
__device__ __forceinline__ void eval_lane(PPtr P, const uint32_t* __restrict__ Acol, CPtr ctr, FPtr full,
                                          const uint32_t* __restrict__ birth, const uint32_t* __restrict__ hb,
                                          const StepC* __restrict__ stepc, const CostK K, uint32_t S, uint32_t S32,
                                          const uint32_t* __restrict__ trow, uint32_t shift, LaneMove& mv)
{
    Windows wn;
    uint32_t todo = lane_windows<GROW>(P + (size_t)mv.u * S32, P + (size_t)((mv.pk & 1u) ? mv.v : mv.u) * S32, Acol, full, birth, S,
                                       S32, mv, wn);
    int delta = 0;
    while (todo) {
        const uint32_t k = __ffs(todo) - 1;
        todo &= todo - 1;
        const uint32_t t = wn.s0 + k - 1;
        delta += item_delta<GROW>(wn, k, ctr[t], GROW ? hb[t] : 0u, __ldg(stepc + t), K);
    }
    mv.delta = delta;
    mv.acc = metropolis(delta, mv.w, trow, shift);
}

// N queue items per lane, items base + 32 r + lane: the cost change of one step of one proposal each, added to the
// proposal's sum.
template <bool GROW, bool ASMEM, int N>
__device__ __forceinline__ void eval_items(const ChainView cv, const StepC* __restrict__ stepc, const CostK K, uint32_t S,
                                           uint32_t base, uint32_t count, uint32_t lane)
{
    int d[N];
    uint32_t slot[N];
    bool live[N];
#pragma unroll
    for (int r = 0; r < N; ++r) {
        const uint32_t g = base + 32 * r + lane;
        live[r] = g < count;
        const uint32_t item = live[r] ? cv.queue[g] : 1u;         // a dead lane works on (proposal 0, bit 1) and drops it
        slot[r] = item >> 5;
        const uint32_t k = item & 31u;
        const uint4 w0 = cv.win[slot[r] * 2], w1 = cv.win[slot[r] * 2 + 1];
        Windows wn;
        wn.Wu = w0.x; wn.Wv = w0.y; wn.Nu = w0.z; wn.Nv = w0.w; wn.Au = w1.x; wn.Av = w1.y; wn.s0 = w1.z;
        wn.born = w1.w;
        const uint32_t t = min(wn.s0 + k - 1, S - 1);
        const StepC sc = ASMEM ? stepc[t] : __ldg(stepc + t);
        d[r] = item_delta<GROW>(wn, k, cv.ctr[t], GROW ? cv.hb[t] : 0u, sc, K);
    }
#pragma unroll
    for (int r = 0; r < N; ++r)
        if (live[r] && d[r]) atomicAdd(cv.acc + slot[r], d[r]);
}

// Evaluation of the proposals named by `need` (one mask per proposal row), shared by the warp: every lane
// prepares its own proposals, the (proposal, step) pairs whose cost changes are queued in shared memory, and
// the warp works the queue off 32 pairs at a time, so that lanes with short and long proposals carry the
// same load.
// ALL: every lane prepares its proposal whether `need` names it or not (its items are dropped if not), so that this
// part is straight-line code; `side_work` is then scheduled into it by the compiler (the draw of the next batch: a
// long chain of dependent integer operations that fills the issue slots the window loads leave empty).
template <bool GROW, bool ASMEM, bool ALL, bool COW, typename SideWork>
__device__ __forceinline__ void eval_batch(const ChainView cv, const uint32_t* __restrict__ Acol,
                                           const uint32_t* __restrict__ birth,
                                           const StepC* __restrict__ stepc, const CostK K, uint32_t S, uint32_t S32,
                                           const uint32_t* __restrict__ trow, uint32_t shift, uint32_t split_at,
                                           const uint32_t (&need)[kMPL], uint32_t lane, LaneMove (&mv)[kMPL],
                                           SideWork&& side_work)
{
    uint32_t todo[kMPL], cnt = 0;
#pragma unroll
    for (int h = 0; h < kMPL; ++h) {
        todo[h] = 0;
        const bool named = (need[h] >> lane) & 1u;
        if (ALL || named) {
            const uint32_t slot = h * 32 + lane;
            Windows wn;
            const uint32_t tm = lane_windows<GROW>(cv.col<COW>(mv[h].u), cv.col<COW>((mv[h].pk & 1u) ? mv[h].v : mv[h].u), Acol, cv.full,
                                                   birth, S, S32, mv[h], wn);
            todo[h] = named ? tm : 0u;
            cv.win[slot * 2] = make_uint4(wn.Wu, wn.Wv, wn.Nu, wn.Nv);
            cv.win[slot * 2 + 1] = make_uint4(wn.Au, wn.Av, wn.s0, wn.born);
            cv.acc[slot] = 0;
        }
        cnt += __popc(todo[h]);
    }
    side_work();
    // exclusive prefix sum of cnt over the lanes, bit-sliced: the five ballots do not depend on one another
    uint32_t pos = 0, total = 0;
    const uint32_t below = (1u << lane) - 1u;
#pragma unroll
    for (int bit = 0; bit < 5 + (kMPL > 1 ? 1 : 0) + (kMPL > 2 ? 1 : 0); ++bit) {
        const uint32_t has = __ballot_sync(0xFFFFFFFFu, (cnt >> bit) & 1u);
        pos += __popc(has & below) << bit;
        total += __popc(has) << bit;
    }
    // queue the set bits of every mask of the lanes named by `pushing`; all 31 positions are tried so that no lane
    // waits on a serial bit scan. Item `first` goes to queue position 0.
    auto push = [&](bool pushing, uint32_t first) {
#pragma unroll
        for (int h = 0; h < kMPL; ++h) {
            const uint32_t td = pushing ? todo[h] : 0u;
            if (__any_sync(0xFFFFFFFFu, td != 0)) {
#pragma unroll
                for (uint32_t k = 1; k < 32; ++k) {
                    const uint32_t bit = (td >> k) & 1u;
                    if (bit) cv.queue[pos - first] = (uint16_t)(((h * 32 + lane) << 5) | k);
                    pos += bit;
                }
            }
        }
        __syncwarp();
    };
    // two items per lane and trip (the two evaluations are independent and overlap), one where 32 or fewer are left
    auto work_off = [&](uint32_t count) {
        for (uint32_t base = 0; base < count; base += 64) {
            if (base + 32 < count) eval_items<GROW, ASMEM, 2>(cv, stepc, K, S, base, count, lane);
            else eval_items<GROW, ASMEM, 1>(cv, stepc, K, S, base, count, lane);
        }
    };
    if (!ASMEM || total <= split_at) {
        push(true, 0u);
        work_off(total);
    } else {
        // ASMEM: the queue holds kQueueCap / 2 items, the worst case of 16 lanes. A batch with more (rare) goes in two
        // halves, lanes 0..15 first.
        const uint32_t mid = __shfl_sync(0xFFFFFFFFu, pos, 16);   // items of lanes 0..15
        push(lane < 16, 0u);
        work_off(mid);
        __syncwarp();
        push(lane >= 16, mid);
        work_off(total - mid);
    }
    __syncwarp();
#pragma unroll
    for (int h = 0; h < kMPL; ++h)
        if ((need[h] >> lane) & 1u) {
            mv[h].delta = cv.acc[h * 32 + lane];
            mv[h].acc = metropolis(mv[h].delta, mv[h].w, trow, shift);
        }
}

// Apply the proposal in window slot `slot` (pk, u, v given): all lanes take part, lane j updates the counters
// of window bit j, lanes 0 and 1 rewrite the words of the schedule and of the full-step bitmap.
template <bool GROW, bool COW>
__device__ __forceinline__ void apply_move(const ChainView cv, uint32_t S, uint32_t S32, uint32_t cap, uint32_t lane,
                                           uint32_t slot, uint32_t pk, uint32_t u, uint32_t v)
{
    const uint4 w0 = cv.win[slot * 2], w1 = cv.win[slot * 2 + 1];
    const uint32_t Wu = w0.x, Wv = w0.y, Nu = w0.z, Nv = w0.w, Au = w1.x, Av = w1.y;
    const bool swap = pk & 1u;
    const uint32_t len = (pk >> 1) & 63u, s0 = pk >> 8;
    const uint32_t run = min(s0 + len, S) - s0;
    const uint32_t nl = min(s0 + len, S - 1) - s0 + 1;
    const bool valid = lane >= 1 && lane <= nl;
    const uint32_t j = valid ? lane : 1u, t = s0 + j - 1;
    const uint32_t pu = (Wu >> j) & 1u, qu = (Wu >> (j - 1)) & 1u, npu = (Nu >> j) & 1u, nqu = (Nu >> (j - 1)) & 1u;
    const uint32_t pv = (Wv >> j) & 1u, qv = (Wv >> (j - 1)) & 1u, npv = (Nv >> j) & 1u, nqv = (Nv >> (j - 1)) & 1u;
    const uint32_t au = (Au >> j) & 1u, av = (Av >> j) & 1u;
    uint4 c = cv.ctr[t];
    c.x += (au & npu) - (au & pu) + (av & npv) - (av & pv);
    if (GROW) {
        const uint32_t mu = (w1.w & 255u) == j ? 0u : 1u, mw = ((w1.w >> 8) & 255u) == j ? 0u : 1u;
        c.y += mu * ((npu & ~nqu) - (pu & ~qu)) + mw * ((npv & ~nqv) - (pv & ~qv));
        const uint32_t dh = (1u - mu) * (npu - pu) + (1u - mw) * (npv - pv);
        if (valid && dh) cv.hb[t] += dh;
    } else {
        c.y += (npu & ~nqu) - (pu & ~qu) + (npv & ~nqv) - (pv & ~qv);
    }
    c.z += (~npu & nqu & 1u) - (~pu & qu & 1u) + (~npv & nqv & 1u) - (~pv & qv & 1u);
    c.w += npu - pu + npv - pv;
    if (valid) cv.ctr[t] = c;
    uint32_t F = __ballot_sync(0xFFFFFFFFu, valid && c.w == cap);   // bit j <-> window bit j
    uint32_t V = __ballot_sync(0xFFFFFFFFu, valid);
    cv.own<COW>(u, lane);
    if (swap) cv.own<COW>(v, lane);
    if (lane < 2) {
        uint32_t M = ((1u << run) - 1u) << 1, NU = Nu, NV = Nv, sbit = s0 - 1;
        if (s0 == 0) { F >>= 1; V >>= 1; M >>= 1; NU >>= 1; NV >>= 1; sbit = 0; }
        const uint32_t wj = (sbit >> 5) + lane, sh = sbit & 31u;
        if (wj < S32 && (lane == 0 || sh != 0)) {
            // lane 0 holds the part of the window that falls into the first word, lane 1 the spill-over
            const uint32_t Vx = lane ? V >> (32 - sh) : V << sh, Fx = lane ? F >> (32 - sh) : F << sh;
            const uint32_t Mx = lane ? M >> (32 - sh) : M << sh;
            const uint32_t NUx = lane ? NU >> (32 - sh) : NU << sh, NVx = lane ? NV >> (32 - sh) : NV << sh;
            if (Vx) cv.full[wj] = (cv.full[wj] & ~Vx) | (Fx & Vx);
            if (Mx) {
                const size_t iu = (size_t)u * S32 + wj;
                cv.P[iu] = (cv.P[iu] & ~Mx) | (NUx & Mx);
                if (swap) {
                    const size_t iv = (size_t)v * S32 + wj;
                    cv.P[iv] = (cv.P[iv] & ~Mx) | (NVx & Mx);
                }
            }
        }
    }
    __syncwarp();
}

// A group of nthr threads (one or more whole warps, this thread being number tid) copies n words. A chain in global
// scratch starts by copying tens of megabytes this way, so eight 16-byte loads per thread are in flight before the
// first store.
__device__ __forceinline__ void copy_words(uint32_t* __restrict__ dst, const uint32_t* __restrict__ src, size_t n,
                                           uint32_t tid, uint32_t nthr = 32)
{
    if ((n & 3) == 0 && ((reinterpret_cast<uintptr_t>(dst) | reinterpret_cast<uintptr_t>(src)) & 15) == 0) {
        uint4* __restrict__ d4 = reinterpret_cast<uint4*>(dst);
        const uint4* __restrict__ s4 = reinterpret_cast<const uint4*>(src);
        const size_t n4 = n / 4;
        size_t i = tid;
        for (; i + 7 * (size_t)nthr < n4; i += 8 * (size_t)nthr) {
            uint4 v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = s4[i + (size_t)nthr * j];
#pragma unroll
            for (int j = 0; j < 8; ++j) d4[i + (size_t)nthr * j] = v[j];
        }
        for (; i < n4; i += nthr) d4[i] = s4[i];
    } else {
        for (size_t i = tid; i < n; i += nthr) dst[i] = src[i];
    }
}

// The copies off the hot path (a bucket fetched into a slice, a best state saved) as one function each, so that the
// chain loop stays small enough for the instruction cache.
__device__ __noinline__ void copy_words_cold(uint32_t* dst, const uint32_t* src, size_t n, uint32_t lane)
{
    copy_words(dst, src, n, lane);
}

// Schedules in global scratch are copy-on-write overlays of the one initial schedule that all chains share: the
// units come in buckets of 2^shift consecutive units, a chain's slice holds a bucket only once the chain has
// rewritten a unit of it, and a bitmap in shared memory says which. Chains change few of their units, so nearly
// every placement window is read from the shared initial schedule, which stays in L2, and not from a private slice
// that only DRAM can hold; a chain that rewrites everything ends up copying its whole slice once, bucket by bucket.
// The bitmap takes the shared memory that a full CTA of chains leaves free (kCowBitsMin to kCowBitsMax buckets): a
// chain of a million moves rewrites thousands of units, and every read of a bucket it owns misses L2, so the buckets
// should be small (with 8192 buckets of 512 units a chain of the largest configuration owned two thirds of them at
// its end; with 40,960 of 64 units it owns an eighth).
constexpr uint32_t kCowBitsMin = 8192, kCowBitsMax = 65536;

// A whole schedule out of a copy-on-write slice: the buckets the slice holds from it, the rest from the initial one.
__device__ __forceinline__ void copy_merged(uint32_t* __restrict__ dst, const uint32_t* __restrict__ mine,
                                            const uint32_t* __restrict__ p0, const uint32_t* have, uint32_t shift,
                                            uint32_t U, uint32_t S32, uint32_t lane)
{
    const uint32_t nb = (U + (1u << shift) - 1u) >> shift;
    for (uint32_t b = 0; b < nb; ++b) {
        const size_t lo = (size_t)(b << shift) * S32, hi = (size_t)min(U, (b + 1u) << shift) * S32;
        const uint32_t* src = (have[b >> 5] >> (b & 31u)) & 1u ? mine : p0;
        copy_words_cold(dst + lo, src + lo, hi - lo, lane);
    }
}

// Hand-over block of a chain that is served by more than one warp (shared memory, one per chain).
// The warps of a chain take the batches in turn: warp w owns batches w, w + W, w + 2W, ... It evaluates a batch
// against whatever state it finds (another warp may be committing an earlier batch meanwhile), then waits for its
// turn, evaluates again the proposals that a move applied in the meantime could have touched, and commits. `turn`
// is the index of the batch whose owner may commit; `napplied` counts the state-changing moves of the chain and
// `applog` keeps the step ranges of the latest kLog of them. The chain-wide scalars are read and written back only
// in a turn that applies a move, starts a temperature level or ends the chain; the two counters that change in
// nearly every batch are kept per warp and added up at the end.
constexpr uint32_t kLog = 16;
constexpr int kMaxW = 2;
struct ChainShare {
    uint64_t cur, best, best_move, best_at_boundary, n_chg, hash;
    uint64_t n_acc[kMaxW], n_inf[kMaxW];
    uint32_t ulen, snap_dirty, stopped, pad;
    uint32_t turn, napplied, pad2[2];
    uint32_t applog[kLog];       // s0 | (s0 + len) << 16 of an applied move
};
constexpr uint32_t kShareSlots4 = (sizeof(ChainShare) + 15) / 16;
// per warp: windows, sums, work queue
__host__ __device__ constexpr uint32_t priv_slots4(bool halfq)
{
    return kWinSlots4 + kAccSlots4 + (halfq ? kHalfQueueSlots4 : kQueueSlots4);
}
// A wait for the turn gives up after this many polls (each at least some tens of nanoseconds apart): the chain then
// reports KVP_ERR_TIMEOUT instead of holding the GPU. A turn lasts microseconds.
constexpr uint32_t kTurnPolls = 1u << 24;

__device__ __forceinline__ uint32_t ld_volatile_u32(const uint32_t* p) { return *reinterpret_cast<const volatile uint32_t*>(p); }
__device__ __forceinline__ void st_volatile_u32(uint32_t* p, uint32_t v) { *reinterpret_cast<volatile uint32_t*>(p) = v; }

// shared-memory words (as uint4 slots) of one chain besides its schedule
// cow4: uint4 slots of the bucket bitmap of a copy-on-write slice (schedules in global scratch), else 0
__host__ __device__ inline uint32_t chain_fixed4(uint32_t S, uint32_t S32, bool grow, uint32_t W, bool halfq, uint32_t cow4)
{
    return S + (S32 + 3) / 4 + (grow ? (S + 3) / 4 : 0u) + cow4 + (W > 1 ? kShareSlots4 : 0u) + W * priv_slots4(halfq);
}

// ASMEM (only with PSMEM): the access bitmap and the per-step constants, which every chain of the CTA reads, are
// staged in shared memory once per CTA. With the schedules in shared memory the L1 cache is down to its minimum and
// cannot hold them.
// Without PSMEM the chain's slice of global scratch is a copy-on-write overlay of the initial schedule when
// prm.cow_slots4 is set (jobs whose slices add up to gigabytes: the chains then start without copying anything), else a
// plain copy of it (small slices: the copy costs nothing and an applied move is cheaper without the take-over).
template <bool PSMEM, bool GROW, int W, bool ASMEM, bool COW>
__global__ void __launch_bounds__(512)
chain_kernel(const ChainParams prm)
{
    static_assert(!COW || !PSMEM, "overlays only for schedules in global scratch");
    static_assert(W >= 1 && W <= kMaxW && (W & (W - 1)) == 0, "warps per chain");
    static_assert(PSMEM || !ASMEM, "shared access bitmap only beside shared schedules");
    extern __shared__ uint4 smem4[];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t cpb = (blockDim.x >> 5) / W;                   // chains per CTA
    const uint32_t cic = warp / W, sub = warp % W;                // chain within the CTA, warp within the chain
    const uint32_t tid = sub * 32 + lane;                         // thread within the chain
    const uint32_t slot = blockIdx.x * cpb + cic;
    const bool active = slot < prm.chain_count;
    if (W == 1 && !ASMEM && !active) return;
    const uint32_t chain = prm.chain_first + slot;
    const uint32_t S = prm.S, S32 = prm.S32, U = prm.U;
    const size_t pwords = (size_t)U * S32;
    const uint32_t f4 = (S32 + 3) / 4;                            // uint4 slots of the full-step bitmap
    const uint32_t h4 = GROW ? (S + 3) / 4 : 0u;                  // uint4 slots of the written-to-HBM counts
    const uint32_t o4 = COW ? prm.cow_slots4 : 0u;                 // the slice is a copy-on-write overlay
    const uint32_t fixed4 = chain_fixed4(S, S32, GROW, W, ASMEM, o4);
    uint4* const mine4 = smem4 + (size_t)cic * fixed4;
    ChainView cv;
    cv.ctr = mine4;
    cv.full = reinterpret_cast<uint32_t*>(mine4 + S);
    cv.hb = reinterpret_cast<uint32_t*>(mine4 + S + f4);
    uint32_t* const cowmap = reinterpret_cast<uint32_t*>(mine4 + S + f4 + h4);   // buckets the slice holds
    ChainShare* const sh = reinterpret_cast<ChainShare*>(mine4 + S + f4 + h4 + o4);
    uint4* const priv4 = mine4 + S + f4 + h4 + o4 + (W > 1 ? kShareSlots4 : 0u) + sub * priv_slots4(ASMEM);
    cv.win = priv4;
    cv.acc = reinterpret_cast<int*>(priv4 + kWinSlots4);
    cv.queue = reinterpret_cast<uint16_t*>(priv4 + kWinSlots4 + kAccSlots4);
    uint32_t* const pool = reinterpret_cast<uint32_t*>(smem4 + (size_t)cpb * fixed4);   // schedules, then A, then constants
    cv.P = PSMEM ? pool + (size_t)cic * pwords : prm.ws + (size_t)slot * pwords;
    cv.p0 = prm.Pcol0; cv.have = COW ? cowmap : nullptr; cv.shared_chain = W > 1; cv.shift = prm.cow_shift; cv.U = U; cv.S32 = S32;
    const uint32_t* Acol = prm.Acol;
    const StepC* stepc = prm.stepc;
    if (ASMEM) {
        const size_t a_off = ((size_t)cpb * pwords + 3) & ~(size_t)3, c_off = (a_off + pwords + 3) & ~(size_t)3;
        uint32_t* const a_s = pool + a_off;
        StepC* const c_s = reinterpret_cast<StepC*>(pool + c_off);
        copy_words(a_s, prm.Acol, pwords, threadIdx.x, blockDim.x);
        for (uint32_t i = threadIdx.x; i < S; i += blockDim.x) c_s[i] = __ldg(prm.stepc + i);
        Acol = a_s;
        stepc = c_s;
    }
    if (active) {
        for (uint32_t i = tid; i < S; i += 32 * W) cv.ctr[i] = __ldg(prm.counters0 + i);
        for (uint32_t i = tid; i < S32; i += 32 * W) cv.full[i] = __ldg(prm.full0 + i);
        if (GROW)
            for (uint32_t i = tid; i < S; i += 32 * W) cv.hb[i] = __ldg(prm.hb0 + i);
        for (uint32_t i = lane; i < kWinSlots4; i += 32) cv.win[i] = make_uint4(0u, 0u, 0u, 0u);
        if (!COW) copy_words(cv.P, prm.Pcol0, pwords, tid, 32 * W);
        else
            for (uint32_t i = tid; i < prm.cow_slots4 * 4; i += 32 * W) cowmap[i] = 0u;   // the slice holds nothing yet
        if (W > 1 && tid == 0) {
            sh->cur = sh->best = sh->best_at_boundary = prm.init_ticks;
            sh->best_move = ~0ull; sh->n_chg = 0; sh->hash = 0;
            for (int w = 0; w < kMaxW; ++w) { sh->n_acc[w] = 0; sh->n_inf[w] = 0; }
            sh->ulen = 0u; sh->snap_dirty = 0u; sh->stopped = 0u; sh->turn = 0u; sh->napplied = 0u;
        }
    }
    if (W > 1 || ASMEM) {
        __syncthreads();
        if (!active) return;
    } else {
        __syncwarp();
    }
    uint32_t* snap = prm.snap ? prm.snap + (size_t)slot * pwords : nullptr;
    uint64_t* ulog = prm.undo_log ? prm.undo_log + (size_t)slot * prm.undo_cap : nullptr;

    // Chain-wide scalars. One warp: they live in registers. Several warps: the master copy is in `sh`; a warp
    // fetches it (`have`) in a turn that needs it and writes it back before it passes the turn on.
    uint64_t cur = prm.init_ticks, best = cur, best_move = ~0ull, best_at_boundary = cur;
    uint64_t n_chg = 0, hash = 0;
    bool snap_dirty = false;                                      // the best state is the current one, not yet saved
    uint32_t ulen = 0;                                            // moves applied since the best state
    uint64_t n_acc = 0, n_inf = 0;                                // this warp's share of the two counters
    uint32_t napp = 0;                                            // state-changing moves so far (W > 1)
    bool have = W == 1;
    auto fetch = [&]() {
        if (W > 1 && !have) {
            cur = sh->cur; best = sh->best; best_move = sh->best_move; best_at_boundary = sh->best_at_boundary;
            n_chg = sh->n_chg; hash = sh->hash; ulen = sh->ulen; snap_dirty = sh->snap_dirty != 0;
            have = true;
        }
    };
    // Ends this warp's turn for batch b: scalars back to `sh` if they were fetched, then the next batch may commit.
    auto pass_turn = [&](uint32_t b) {
        __syncwarp();
        if (lane == 0) {
            if (have) {
                sh->cur = cur; sh->best = best; sh->best_move = best_move; sh->best_at_boundary = best_at_boundary;
                sh->n_chg = n_chg; sh->hash = hash; sh->ulen = ulen; sh->snap_dirty = snap_dirty ? 1u : 0u;
            }
            sh->n_acc[sub] = n_acc; sh->n_inf[sub] = n_inf;
            __threadfence_block();
            if (!(prm.drop_first_turn && b == 0)) st_volatile_u32(&sh->turn, b + 1u);
        }
        have = false;
    };

    uint64_t lvl_start = 0;                                       // first move of the level
    uint32_t base = 0;                                            // index of the level's first batch (mod 2^32)
    bool stop = false;
    for (uint32_t level = 0; level < prm.levels && lvl_start < prm.upto; ++level) {
        // a temperature level: its moves in batches of up to 32 * kMPL consecutive moves (fewer than 2^32 batches:
        // the host refuses longer levels)
        const uint64_t lvl_len = (level + 1 < prm.levels ? min(lvl_start + prm.per_level, prm.upto) : prm.upto) - lvl_start;
        const uint32_t nbat = (uint32_t)((lvl_len + kBatch - 1) / kBatch);
        const uint32_t last_nb = (uint32_t)(lvl_len - (uint64_t)(nbat - 1) * kBatch);
        const bool last_level = lvl_start + lvl_len >= prm.upto;
        const uint32_t shift = __ldg(prm.shifts + level);
        const uint32_t* trow = prm.table + (size_t)level * KVP_TABLE_Q;
        if (W == 1 && level > 0) {
            if (prm.early_permille && level >= prm.early_from &&
                (best_at_boundary - best) * 1000ull < best_at_boundary * (uint64_t)prm.early_permille) {
                stop = true;
                break;
            }
            best_at_boundary = best;
        }
        // A batch: move m + 32 h + lane in row h of its lane. Every lane draws and evaluates its own proposals
        // against the current state; the warp then commits them in move order. A move that changes the schedule
        // invalidates only later moves whose step windows overlap its own; those are evaluated again before their
        // turn comes, so the outcome is that of the sequential chain.
        bool have_next = false;                                   // `next` holds the draw of the batch about to start
        LaneMove next;
        next.pk = next.u = next.v = next.w = 0u; next.delta = 0; next.inf = next.acc = next.chg = false;
        for (uint32_t bi = (sub - base) & (W - 1); bi < nbat; bi += W) {
            const uint64_t m = lvl_start + (uint64_t)bi * kBatch;
            const uint32_t nb = bi + 1 < nbat ? kBatch : last_nb;
            const uint32_t b = base + bi;
            uint32_t n0 = 0;
            if (W > 1) {
                // Moves applied from now on may be half visible to the reads below: they are checked for at the turn.
                n0 = __shfl_sync(0xFFFFFFFFu, ld_volatile_u32(&sh->napplied), 0);
                __threadfence_block();
            }
            static_assert(kMPL == 1, "the draw of the next batch is carried in one LaneMove");
            LaneMove mv[kMPL];
            uint32_t todo[kMPL], need[kMPL];
            if (have_next) {
                mv[0] = next;
            } else {
                uint32_t r[4];
                const uint64_t mine = m + lane;
                philox4x32_10((uint32_t)mine, (uint32_t)(mine >> 32), chain, TAG_MOVE, prm.keys, r);
                decode_move(r, prm.p_swap_256, prm.len_choices, S, U, mv[0]);
            }
            mv[0].inf = false; mv[0].acc = false; mv[0].chg = false; mv[0].delta = 0;
            todo[0] = nb >= 32 ? 0xFFFFFFFFu : (1u << nb) - 1u;
            need[0] = todo[0];
            // the proposals of this warp's next batch of the level are drawn while this batch's windows are loaded
            // (drawn, and dropped, even where the level has no further batch for this warp)
            eval_batch<GROW, ASMEM, true, COW>(cv, Acol, prm.birth, stepc, prm.K, S, S32, trow, shift, prm.split_at, need, lane, mv,
                                          [&]() {
                                              uint32_t r[4];
                                              const uint64_t mine = m + (uint64_t)W * kBatch + lane;
                                              philox4x32_10((uint32_t)mine, (uint32_t)(mine >> 32), chain, TAG_MOVE, prm.keys, r);
                                              decode_move(r, prm.p_swap_256, prm.len_choices, S, U, next);
                                          });
            have_next = bi + W < nbat;
#pragma unroll
            for (int h = 0; h < kMPL; ++h) need[h] = 0;
            if (W > 1) {
                // wait for the turn
                uint32_t polls = 0, t;
                for (;;) {
                    t = __shfl_sync(0xFFFFFFFFu, ld_volatile_u32(&sh->turn), 0);
                    if (t == b || ++polls > kTurnPolls) break;
                    __nanosleep(64);
                }
                __threadfence_block();
                if (t != b) {                                     // gave up: flag it, let the others pass, leave
                    if (lane == 0) {
                        atomicExch(prm.err, 1u);
                        st_volatile_u32(&sh->stopped, 2u);
                        __threadfence_block();
                        st_volatile_u32(&sh->turn, b + 1u);
                    }
                    return;
                }
                if (ld_volatile_u32(&sh->stopped)) {              // the chain has ended: pass the turn on and leave
                    __syncwarp();
                    if (lane == 0) st_volatile_u32(&sh->turn, b + 1u);
                    return;
                }
                napp = sh->napplied;
                // proposals whose steps meet those of a move applied since this batch was evaluated
                if (napp - n0 > kLog) {
#pragma unroll
                    for (int h = 0; h < kMPL; ++h) need[h] = todo[h];
                } else {
                    for (uint32_t k = n0; k != napp; ++k) {
                        const uint32_t e = sh->applog[k % kLog], s0b = e & 0xFFFFu, endb = e >> 16;
#pragma unroll
                        for (int h = 0; h < kMPL; ++h) {
                            const uint32_t s0 = mv[h].pk >> 8, end = s0 + ((mv[h].pk >> 1) & 63u);
                            need[h] |= __ballot_sync(0xFFFFFFFFu, s0 <= endb + 1 && s0b <= end) & todo[h];
                        }
                    }
                }
                if (bi == 0 && level > 0) {                       // the level's first batch: stop rule, new reference
                    fetch();
                    if (prm.early_permille && level >= prm.early_from &&
                        (best_at_boundary - best) * 1000ull < best_at_boundary * (uint64_t)prm.early_permille) {
                        stop = true;
                        break;
                    }
                    best_at_boundary = best;
                }
            }
            for (;;) {
                uint32_t any_need = 0;
#pragma unroll
                for (int h = 0; h < kMPL; ++h) any_need |= need[h];
                if (any_need)
                    eval_batch<GROW, ASMEM, false, COW>(cv, Acol, prm.birth, stepc, prm.K, S, S32, trow, shift, prm.split_at, need, lane, mv,
                                                   []() {});
                bool applied = false;
#pragma unroll
                for (int h = 0; h < kMPL; ++h) need[h] = 0;
#pragma unroll
                for (int h = 0; h < kMPL; ++h) {
                    if (applied || !todo[h]) continue;
                    const uint32_t infb = __ballot_sync(0xFFFFFFFFu, mv[h].inf);
                    const uint32_t accb = __ballot_sync(0xFFFFFFFFu, !mv[h].inf && mv[h].acc);
                    const uint32_t blk = __ballot_sync(0xFFFFFFFFu, !mv[h].inf && mv[h].acc && mv[h].chg) & todo[h];
                    if (!blk) {                                   // nothing in this row changes the schedule
                        n_inf += __popc(infb & todo[h]);
                        n_acc += __popc(accb & todo[h]);
                        todo[h] = 0;
                        continue;
                    }
                    const uint32_t bb = __ffs(blk) - 1;
                    const uint32_t done = todo[h] & (0xFFFFFFFFu >> (31 - bb));  // the row's moves up to and including bb
                    n_inf += __popc(infb & done);
                    n_acc += __popc(accb & done);
                    fetch();
                    ++n_chg;
                    const int delta = __shfl_sync(0xFFFFFFFFu, mv[h].delta, bb);
                    const uint32_t pk = __shfl_sync(0xFFFFFFFFu, mv[h].pk, bb);
                    const uint32_t bu = __shfl_sync(0xFFFFFFFFu, mv[h].u, bb), bv = __shfl_sync(0xFFFFFFFFu, mv[h].v, bb);
                    const uint64_t after = (uint64_t)((int64_t)cur + delta);
                    if (snap && snap_dirty && after >= best) {    // leaving the best state: save it first
                        copy_words(snap, cv.P, pwords, lane);
                        snap_dirty = false;
                    }
                    apply_move<GROW, COW>(cv, S, S32, prm.cap, lane, h * 32 + bb, pk, bu, bv);
                    // The applied move rewrote steps s0b .. s0b + len_b (bits, counters, full flags). A later
                    // proposal read steps s0 - 1 .. s0 + len: it has to be evaluated again iff the two ranges meet.
                    const uint32_t s0b = pk >> 8, endb = s0b + ((pk >> 1) & 63u);
                    if (W > 1) {                                  // tell the warps that are evaluating later batches
                        if (lane == 0) {
                            sh->applog[napp % kLog] = s0b | (endb << 16);
                            __threadfence_block();
                            st_volatile_u32(&sh->napplied, napp + 1u);
                        }
                        ++napp;
                    }
                    cur = after;
                    const uint64_t mb = m + 32u * h + bb;
                    hash = (hash ^ mb) * 0x9E3779B97F4A7C15ull + cur;
                    if (cur < best) { best = cur; best_move = mb; snap_dirty = true; ulen = 0; }
                    else if (ulog) {                              // every move is its own inverse: remember it
                        if (ulen < prm.undo_cap && lane == 0) ulog[ulen] = mb;
                        if (ulen <= prm.undo_cap) ++ulen;
                    }
                    todo[h] &= ~done;
#pragma unroll
                    for (int h2 = 0; h2 < kMPL; ++h2) {
                        const uint32_t s0 = mv[h2].pk >> 8, end = s0 + ((mv[h2].pk >> 1) & 63u);
                        need[h2] = __ballot_sync(0xFFFFFFFFu, s0 <= endb + 1 && s0b <= end) & todo[h2];
                    }
                    applied = true;
                }
                if (!applied) break;
            }
            if (W > 1 && !(last_level && bi + 1 == nbat)) pass_turn(b);   // hand the chain to the owner of the next batch
        }
        if (stop) break;                                          // `base` stays the index of the batch that stopped
        base += nbat;
        lvl_start += lvl_len;
    }
    const uint64_t m_end = stop ? lvl_start : prm.upto;           // moves done when the chain ended
    // The warp that committed the last batch, or that ended the chain by the stop rule, reports.
    if (W > 1) {
        const bool writer = stop || (base ? ((base - 1u) & (W - 1)) == sub : sub == 0);
        if (!writer) return;
        fetch();
        sh->n_acc[sub] = n_acc; sh->n_inf[sub] = n_inf;           // all lanes write the same values
        __syncwarp();
        n_acc = 0; n_inf = 0;
        for (int w = 0; w < W; ++w) { n_acc += sh->n_acc[w]; n_inf += sh->n_inf[w]; }
    }
    if (snap && snap_dirty) copy_words(snap, cv.P, pwords, lane);
    if (ulog && lane == 0) prm.undo_len[slot] = ulen;
    if (COW && prm.cow_out)                                    // which buckets the slice holds (for the walk back)
        for (uint32_t i = lane; i < prm.cow_slots4 * 4; i += 32)
            prm.cow_out[(size_t)slot * (prm.cow_slots4 * 4) + i] = cowmap[i];
    if (lane == 0) {
        kvp_chain_result res;
        res.best_ticks = best; res.best_move = best_move; res.final_ticks = cur; res.moves_done = m_end;
        res.n_accepted = n_acc; res.n_changed = n_chg; res.n_infeasible = n_inf; res.traj_hash = hash;
        prm.results[chain - prm.result_base] = res;
    }
    if (prm.dump && slot == 0) {
        __syncwarp();
        if (!COW) copy_words(prm.dump, cv.P, pwords, lane);
        else copy_merged(prm.dump, cv.P, prm.Pcol0, cowmap, prm.cow_shift, U, S32, lane);
    }
    if (W > 1 && stop) {                                          // ended by the stop rule: release the next owner
        __syncwarp();
        if (lane == 0) {
            st_volatile_u32(&sh->stopped, 1u);
            __threadfence_block();
            st_volatile_u32(&sh->turn, base + 1u);
        }
    }
}

// ---------------------------------------------------------------------------------------------------------------
// The wide chain kernel: one warp per chain, kRows proposals per lane, so a batch is 32 * kRows consecutive moves.
//
// Most proposals are settled by the placement bits alone: a swap of two units with equal placement over the run
// changes nothing, a flip into a full step is infeasible (Eq. 5). Every lane first classifies its kRows proposals
// that way (the Philox draws and the window loads of the rows are independent, so the warp has instruction-level
// parallelism where the narrow kernel has none). Only the rest, typically a tenth to a third, needs the access
// windows, the set of steps whose cardinalities change and Eq. 2-4 at those steps: their indices are compacted into
// a list, and the warp works the list off 32 at a time, one proposal per lane, through the shared work queue of
// (proposal, step) items. The commit walks the batch in move order and applies every accepted, state-changing
// proposal it meets until it reaches one whose step range meets that of a move applied since it was evaluated;
// those are evaluated again, all at once, and the walk goes on from there. The outcome is the sequential chain's.
constexpr int kRows = 4;
// Largest CTA of the wide kernel with schedules in global scratch; it sets the registers a thread may use (65,536
// per SM over the resident threads), hence how many chains an SM holds at a time.
#ifndef KVP_WIDE_GLOBAL_THREADS
#define KVP_WIDE_GLOBAL_THREADS 512
#endif
constexpr int kWideGlobalThreads = KVP_WIDE_GLOBAL_THREADS;
constexpr uint32_t kWide = 32 * kRows;
constexpr uint32_t kWideQueueSlots4 = (32 * 31 * 2 + 15) / 16;     // the items of one pass of 32 proposals

template <typename CT> __device__ __forceinline__ uint4 ctr_load(const CT* c, uint32_t t);
template <> __device__ __forceinline__ uint4 ctr_load<uint4>(const uint4* c, uint32_t t) { return c[t]; }
template <> __device__ __forceinline__ uint4 ctr_load<ushort4>(const ushort4* c, uint32_t t)
{
    const ushort4 v = c[t];
    return make_uint4(v.x, v.y, v.z, v.w);
}
template <typename CT> __device__ __forceinline__ void ctr_store(CT* c, uint32_t t, uint4 v);
template <> __device__ __forceinline__ void ctr_store<uint4>(uint4* c, uint32_t t, uint4 v) { c[t] = v; }
template <> __device__ __forceinline__ void ctr_store<ushort4>(ushort4* c, uint32_t t, uint4 v)
{
    c[t] = make_ushort4((unsigned short)v.x, (unsigned short)v.y, (unsigned short)v.z, (unsigned short)v.w);
}

// Where a chain of the wide kernel keeps its state. CT: the four per-step cardinalities as 16-bit fields when the
// schedule lives in shared memory (then units < 2^16), as 32-bit fields otherwise. COW: see above.
template <typename CT, bool COW, int COLV>
struct WideView {
    const uint32_t* p0;          // COW: [U][S32] the initial schedule
    uint32_t* have;              // COW: [cow_slots4 * 4] buckets present in P (shared)
    uint32_t shift, U, S32;      // COW: bucket size; units; words per unit
    __device__ __forceinline__ const uint32_t* col(uint32_t u) const
    {
        if (COW) {
            const uint32_t b = u >> shift;
            return ((have[b >> 5] >> (b & 31u)) & 1u ? P : p0) + (size_t)u * S32;
        }
        return P + (size_t)u * S32;
    }
    // Before unit u is rewritten: its bucket is copied into the slice if it is not there yet (all lanes, u uniform).
    __device__ __forceinline__ void own(uint32_t u, uint32_t lane) const
    {
        if (!COW) return;
        const uint32_t b = u >> shift;
        if ((have[b >> 5] >> (b & 31u)) & 1u) return;
        const size_t lo = (size_t)(b << shift) * S32, hi = (size_t)min(U, (b + 1u) << shift) * S32;
        copy_words(P + lo, p0 + lo, hi - lo, lane);
        __syncwarp();
        if (lane == 0) have[b >> 5] |= 1u << (b & 31u);
        __syncwarp();
    }
    uint32_t* P;                 // [U][S32] schedule, time-packed (shared or global)
    CT* ctr;                     // [S] {hr, mi, mo, occ} (shared)
    uint32_t* full;              // [S32] bit t set iff occ[t] == cap (shared)
    uint32_t* hb;                // growing cache: [S] units written to HBM at birth (shared)
    uint32_t* fnow;              // [S] the present cost of every step, Eq. 2 (shared)
    uint4* win;                  // [kWide][2] by proposal: {pk, u, v, -} until it is evaluated, then its windows
    int* acc;                    // [kWide] by proposal: its cost change being summed
    uint8_t* nt;                 // [kWide] the proposals that need a cost evaluation, compacted
    uint16_t* queue;             // [32 * 31] work items (proposal << 5 | window bit) of one pass
};

// The scalars of a chain that only an applied move or a level boundary touches: in shared memory, so that the loop
// over the batches keeps its registers for the proposals.
struct WideScalars {
    uint64_t cur, best, best_move, best_at_boundary, n_chg, hash;
    uint32_t ulen;               // moves applied since the best state
    uint32_t snap_dirty;         // the best state is the current one and not saved yet
    uint32_t qn;                 // items reserved in the work queue during a pass (0 between passes)
    uint32_t pad;
    // what the chain's evaluations amounted to (kvp_anneal_stats): proposals evaluated again after an applied move,
    // proposals that needed a cost evaluation, (proposal, step) items
    uint64_t n_again, n_listed, n_items;
    uint64_t n_acc, n_inf;       // accepted / infeasible proposals of earlier calls on this state (replica exchange)
    uint64_t pad2;
};
constexpr uint32_t kWideScalars4 = sizeof(WideScalars) / 16;

// the part of wide_fixed4 that outlives a batch (what a replica-exchange run saves between its rounds)
// cow4: uint4 slots of the bucket bitmap (schedules in global scratch)
__host__ __device__ inline uint32_t wide_persist4(uint32_t S, uint32_t S32, bool grow, bool shared, uint32_t cow4)
{
    return (shared ? (S + 1) / 2 : S) + (S32 + 3) / 4 + (grow ? (S + 3) / 4 : 0u) + (S + 3) / 4 + (shared ? 0u : cow4) +
           kWideScalars4;
}

// shared-memory words (as uint4 slots) of one chain of the wide kernel besides its schedule
__host__ __device__ inline uint32_t wide_fixed4(uint32_t S, uint32_t S32, bool grow, bool shared, uint32_t cow4)
{
    return (shared ? (S + 1) / 2 : S) + (S32 + 3) / 4 + (grow ? (S + 3) / 4 : 0u) + (S + 3) / 4 +
           (shared ? 0u : cow4) + kWideScalars4 +
           2 * kWide + kWide / 4 + kWide / 16 + kWideQueueSlots4;
}

// N queue items per lane, items base + 32 r + lane: the cost change of one step of one proposal each, added to the
// proposal's sum.
template <bool GROW, int N, typename CT, bool COW, int COLV>
__device__ __forceinline__ void wide_items(const WideView<CT, COW, COLV> cv, const StepC* __restrict__ stepc, const CostK K, uint32_t S,
                                           uint32_t base, uint32_t count, uint32_t lane)
{
    int d[N];
    uint32_t id[N];
    bool live[N];
#pragma unroll
    for (int r = 0; r < N; ++r) {
        const uint32_t g = base + 32 * r + lane;
        live[r] = g < count;
        const uint32_t item = cv.queue[live[r] ? g : 0u];         // a dead lane repeats item 0 and drops the result
        id[r] = item >> 5;
        const uint32_t k = item & 31u;
        const uint4 w0 = cv.win[id[r] * 2], w1 = cv.win[id[r] * 2 + 1];
        Windows wn;
        wn.Wu = w0.x; wn.Wv = w0.y; wn.Nu = w0.z; wn.Nv = w0.w; wn.Au = w1.x; wn.Av = w1.y; wn.s0 = w1.z;
        wn.born = w1.w;
        const uint32_t t = min(wn.s0 + k - 1, S - 1);
        const StepC sc = stepc[t];
        d[r] = (int)(item_cost_after<GROW>(wn, k, ctr_load<CT>(cv.ctr, t), GROW ? cv.hb[t] : 0u, sc, K) - cv.fnow[t]);
    }
#pragma unroll
    for (int r = 0; r < N; ++r)
        if (live[r] && d[r]) atomicAdd(cv.acc + id[r], d[r]);
}

// Per-lane record of the kRows proposals a lane owns in the current batch. Row h of lane l is move m + 32 h + l.
// inf / acc / chg: one bit per row.
struct WideMoves {
    uint32_t pk[kRows], u[kRows], v[kRows], w[kRows];
    int delta[kRows];
    uint32_t inf, acc, chg;
};

// Second half of evaluating a proposal that is known to change bits and to be feasible: given its placement windows
// (Wu; wv = the window of v for a swap), the access windows, the windows after the move and the set of window bits
// (steps) whose cardinalities, hence cost, change. Same conventions as lane_windows.
template <bool GROW, int COLV>
__device__ __forceinline__ uint32_t changed_steps(uint32_t Wu, uint32_t wv, const uint32_t* __restrict__ Acol,
                                                  const uint32_t* __restrict__ birth, uint32_t S, uint32_t S32,
                                                  uint32_t pk, uint32_t u, uint32_t v, Windows& wn)
{
    const bool swap = pk & 1u;
    const uint32_t len = (pk >> 1) & 63u, s0 = pk >> 8;
    const uint32_t run = min(s0 + len, S) - s0;                   // steps whose placement bits change hands
    const uint32_t nl = min(s0 + len, S - 1) - s0 + 1;            // affected steps: the run and the step after it
    const uint32_t M = ((1u << run) - 1u) << 1;
    const uint32_t Sb = ((1u << nl) - 1u) << 1;
    const WinPos wp = window_pos(S32, s0);
    const uint32_t Au = window_at<COLV>(Acol + (size_t)u * S32, wp);
    const uint32_t av = window_at<COLV>(Acol + (size_t)(swap ? v : u) * S32, wp);   // a flip reads unit u twice
    const uint32_t Av = swap ? av : 0u, Wv = swap ? wv : 0u;
    uint32_t Bu = 0u, Bv = 0u, live = 0xFFFFFFFFu;
    if (GROW) {
        uint32_t Lu, Lv;
        alive_born(__ldg(birth + u), s0, Lu, Bu);
        alive_born(__ldg(birth + (swap ? v : u)), s0, Lv, Bv);
        live = Lu & Lv;
        if (!swap) Bv = 0u;
    }
    const uint32_t D = (swap ? (Wu ^ Wv) : 0xFFFFFFFFu) & M & live;      // bits that toggle
    uint32_t Nu = Wu ^ D, Nv = swap ? (Wv ^ D) : 0u;
    if (s0 == 0) {                                                // the virtual step -1 follows step 0
        Nu = (Nu & ~1u) | ((Nu >> 1) & 1u);
        Nv = (Nv & ~1u) | ((Nv >> 1) & 1u);
    }
    wn.Wu = Wu; wn.Wv = Wv; wn.Nu = Nu; wn.Nv = Nv; wn.Au = Au; wn.Av = Av; wn.s0 = s0;
    wn.born = GROW ? ((Bu ? 31u - __clz(Bu) : 0u) | ((Bv ? 31u - __clz(Bv) : 0u) << 8)) : 0u;
    const uint32_t hr = (Au ^ Av) & (Wu ^ Nu);                    // a hit is won or lost (v mirrors u in a swap)
    const uint32_t euo = (Wu ^ (Wu << 1)) & ~Bu, eun = (Nu ^ (Nu << 1)) & ~Bu;
    const uint32_t evo = (Wv ^ (Wv << 1)) & ~Bv, evn = (Nv ^ (Nv << 1)) & ~Bv;
    const uint32_t mg = (euo ^ eun) | (euo & eun & (Wu ^ Nu)) | (evo ^ evn) | (evo & evn & (Wv ^ Nv));
    const uint32_t wr = ((Wu ^ Nu) & Bu) | ((Wv ^ Nv) & Bv);
    return (hr | mg | wr) & Sb;
}

// First half of an evaluation, placement bits only: a swap of equal placements changes nothing, a flip into a full
// step is infeasible (Eq. 5). The proposals of `need` (per lane: bit h = its row h) that need more are listed in cv.nt
// with their placement windows parked in their slots. `listed`: how many; `mine`: which of this lane's rows.
// ALL: nearly every row is named (a fresh batch): the window loads of all rows are issued before any is used, named
// or not (every row holds a drawn proposal, so every address is good). Otherwise rows without a named proposal are
// skipped.
template <bool GROW, bool ALL, typename CT, bool COW, int COLV>
__device__ __forceinline__ void wide_classify(const WideView<CT, COW, COLV> cv, const uint32_t* __restrict__ birth, uint32_t S,
                                              uint32_t S32, uint32_t need, uint32_t lane, WideMoves& mv, uint32_t& listed,
                                              uint32_t& mine)
{
    const uint32_t below = (1u << lane) - 1u;
    uint32_t Wu[kRows], Wv[kRows], Fw[kRows], Lv[kRows];
    bool skip[kRows];
#pragma unroll
    for (int h = 0; h < kRows; ++h) {
        skip[h] = ALL ? false : !__any_sync(0xFFFFFFFFu, (need >> h) & 1u);
        Wu[h] = Wv[h] = Fw[h] = 0u; Lv[h] = 0xFFFFFFFFu;
        if (skip[h]) continue;                                    // warp-uniform
        const uint32_t pk = mv.pk[h], s0 = pk >> 8;
        const bool swap = pk & 1u;
        const WinPos wp = window_pos(S32, s0);
        Wu[h] = window_at<COLV>(cv.col(mv.u[h]), wp);
        // the second window: the other unit's placement for a swap, the full-step bitmap for a flip
        const uint32_t* second = swap ? cv.col(mv.v[h]) : cv.full;
        const uint32_t w2 = window_at<COLV>(second, wp);
        Wv[h] = swap ? w2 : Wu[h];
        Fw[h] = w2;
        if (GROW) {
            uint32_t La, Lb, Bu, Bv;
            alive_born(__ldg(birth + mv.u[h]), s0, La, Bu);
            alive_born(__ldg(birth + (swap ? mv.v[h] : mv.u[h])), s0, Lb, Bv);
            Lv[h] = La & Lb;
        }
    }
#pragma unroll
    for (int h = 0; h < kRows; ++h) {
        if (skip[h]) continue;
        const bool named = (need >> h) & 1u;
        const uint32_t pk = mv.pk[h];
        const bool swap = pk & 1u;
        const uint32_t len = (pk >> 1) & 63u, s0 = pk >> 8;
        const uint32_t run = min(s0 + len, S) - s0;
        const uint32_t M = ((1u << run) - 1u) << 1;
        const uint32_t D = (swap ? Wu[h] ^ Wv[h] : 0xFFFFFFFFu) & M & Lv[h];   // a flip toggles every bit of the run
        const bool chg = D != 0;
        const bool inf = !swap && (~Wu[h] & D & Fw[h]) != 0;      // a flip may not raise a full step (Eq. 5)
        if (named) {
            const uint32_t bit = 1u << h;
            mv.chg = chg ? mv.chg | bit : mv.chg & ~bit;
            mv.inf = inf ? mv.inf | bit : mv.inf & ~bit;
            mv.acc = inf ? mv.acc & ~bit : mv.acc | bit;          // nothing changes: cost change 0, always accepted
            mv.delta[h] = 0;
        }
        const bool more = named && chg && !inf;
        const uint32_t mb = __ballot_sync(0xFFFFFFFFu, more);
        const uint32_t id = h * 32 + lane;
        // the slot of a proposal that is not listed is not looked at again, so a fresh batch parks every row's
        // windows without a test
        if (ALL || more) {
            cv.win[id * 2] = make_uint4(pk, mv.u[h], mv.v[h], Wu[h]);
            cv.win[id * 2 + 1].x = Wv[h];
            cv.acc[id] = 0;
        }
        if (more) {
            cv.nt[listed + __popc(mb & below)] = (uint8_t)id;
            mine |= 1u << h;
        }
        listed += __popc(mb);
    }
}

// Evaluation of the proposals named by `need` (per lane: bit h = its row h) against the current state.
// fresh: a new batch, nearly every row named (see wide_classify).
template <bool GROW, typename CT, bool COW, int COLV>
__device__ __forceinline__ void wide_evaluate(const WideView<CT, COW, COLV> cv, const uint32_t* __restrict__ Acol,
                                              const uint32_t* __restrict__ birth, const StepC* __restrict__ stepc,
                                              const CostK K, uint32_t S, uint32_t S32, const uint32_t* __restrict__ trow,
                                              uint32_t shift, uint32_t need, bool fresh, uint32_t lane, WideMoves& mv,
                                              WideScalars* sc)
{
    // 1. placement bits only; the proposals that need more are listed
    uint32_t listed = 0;                                          // proposals listed (warp-uniform)
    uint32_t mine = 0;                                            // bit h: this lane's row h is listed
    if (fresh) wide_classify<GROW, true>(cv, birth, S, S32, need, lane, mv, listed, mine);
    else wide_classify<GROW, false>(cv, birth, S, S32, need, lane, mv, listed, mine);
    if (!listed) return;                                          // warp-uniform
    if (lane == 0) sc->n_listed += listed;
    __syncwarp();
    // 2. the listed proposals, 32 at a time, one per lane: access windows, the steps whose cost changes, and those
    //    (proposal, step) items through the shared queue
    for (uint32_t first = 0; first < listed; first += 32) {
        const uint32_t g = first + lane;
        const bool live = g < listed;
        const uint32_t id = cv.nt[live ? g : first];
        const uint4 who = cv.win[id * 2];
        const uint32_t wv = cv.win[id * 2 + 1].x;
        Windows wn;
        const uint32_t tm = changed_steps<GROW, COLV>(who.w, wv, Acol, birth, S, S32, who.x, who.y, who.z, wn);
        __syncwarp();                                             // every lane has read its proposal
        const uint32_t todo = live ? tm : 0u;
        if (live) {
            cv.win[id * 2] = make_uint4(wn.Wu, wn.Wv, wn.Nu, wn.Nv);
            cv.win[id * 2 + 1] = make_uint4(wn.Au, wn.Av, wn.s0, wn.born);
        }
        // every lane reserves room for its items in the queue (the order of the items does not matter)
        const uint32_t cnt = __popc(todo);
        uint32_t pos = cnt ? atomicAdd(&sc->qn, cnt) : 0u;
        __syncwarp();
        const uint32_t total = sc->qn;
        __syncwarp();
        if (total) {
            if (lane == 0) { sc->n_items += total; sc->qn = 0u; }
            if (COW) {
                // many chains per SM, issue slots scarce: every lane peels its own set bits, highest first (the order
                // of the items in the queue does not matter: their cost changes are summed)
                for (uint32_t td = todo; td != 0u;) {
                    const uint32_t k = 31u - __clz(td);
                    cv.queue[pos++] = (uint16_t)((id << 5) | k);
                    td ^= 1u << k;
                }
            } else {
                // few chains per SM, latency scarce: all 31 positions tried, no lane waits on a serial bit scan
#pragma unroll
                for (uint32_t k = 1; k < 32; ++k) {
                    const uint32_t bit = (todo >> k) & 1u;
                    if (bit) cv.queue[pos] = (uint16_t)((id << 5) | k);
                    pos += bit;
                }
            }
            __syncwarp();
            for (uint32_t base = 0; base < total; base += 64) {
                if (base + 32 < total) wide_items<GROW, 2>(cv, stepc, K, S, base, total, lane);
                else wide_items<GROW, 1>(cv, stepc, K, S, base, total, lane);
            }
        }
        __syncwarp();
    }
    // 3. the owners take the sums and decide. Straight-line over the rows (the sums and the thresholds of all rows
    //    are loaded before any is used); a row that is not listed reads a stale sum and drops the outcome.
    int d[kRows];
    uint32_t thr[kRows];
#pragma unroll
    for (int h = 0; h < kRows; ++h) d[h] = cv.acc[h * 32 + lane];
#pragma unroll
    for (int h = 0; h < kRows; ++h) {
        const uint32_t q = (uint32_t)max(d[h], 0) >> shift;
        thr[h] = __ldg(trow + min(q, (uint32_t)KVP_TABLE_Q - 1u));
        if (q >= KVP_TABLE_Q) thr[h] = 0u;                        // beyond the table: never accepted
    }
#pragma unroll
    for (int h = 0; h < kRows; ++h) {
        const bool lst = (mine >> h) & 1u;
        const bool ok = d[h] <= 0 || mv.w[h] < thr[h];            // quantised exp(-delta/C), as in metropolis()
        const uint32_t bit = 1u << h;
        if (lst) {
            mv.delta[h] = d[h];
            mv.acc = ok ? mv.acc | bit : mv.acc & ~bit;
        }
    }
}

// Apply the proposal whose windows are in slot `id` (pk, u, v given): all lanes take part, lane j updates the
// counters of window bit j, lanes 0 and 1 rewrite the words of the schedule and of the full-step bitmap.
template <bool GROW, typename CT, bool COW, int COLV>
__device__ __forceinline__ void wide_apply(const WideView<CT, COW, COLV> cv, const StepC* __restrict__ stepc, const CostK K,
                                           uint32_t S, uint32_t S32, uint32_t cap, uint32_t lane,
                                           uint32_t id, uint32_t pk, uint32_t u, uint32_t v)
{
    const uint4 w0 = cv.win[id * 2], w1 = cv.win[id * 2 + 1];
    const uint32_t Wu = w0.x, Wv = w0.y, Nu = w0.z, Nv = w0.w, Au = w1.x, Av = w1.y;
    const bool swap = pk & 1u;
    const uint32_t len = (pk >> 1) & 63u, s0 = pk >> 8;
    const uint32_t run = min(s0 + len, S) - s0;
    const uint32_t nl = min(s0 + len, S - 1) - s0 + 1;
    const bool valid = lane >= 1 && lane <= nl;
    const uint32_t j = valid ? lane : 1u, t = s0 + j - 1;
    const uint32_t pu = (Wu >> j) & 1u, qu = (Wu >> (j - 1)) & 1u, npu = (Nu >> j) & 1u, nqu = (Nu >> (j - 1)) & 1u;
    const uint32_t pv = (Wv >> j) & 1u, qv = (Wv >> (j - 1)) & 1u, npv = (Nv >> j) & 1u, nqv = (Nv >> (j - 1)) & 1u;
    const uint32_t au = (Au >> j) & 1u, av = (Av >> j) & 1u;
    uint4 c = ctr_load<CT>(cv.ctr, t);
    uint32_t hbn = 0u;
    c.x += (au & npu) - (au & pu) + (av & npv) - (av & pv);
    if (GROW) {
        const uint32_t mu = (w1.w & 255u) == j ? 0u : 1u, mw = ((w1.w >> 8) & 255u) == j ? 0u : 1u;
        c.y += mu * ((npu & ~nqu) - (pu & ~qu)) + mw * ((npv & ~nqv) - (pv & ~qv));
        const uint32_t dh = (1u - mu) * (npu - pu) + (1u - mw) * (npv - pv);
        hbn = cv.hb[t] + dh;
        if (valid && dh) cv.hb[t] = hbn;
    } else {
        c.y += (npu & ~nqu) - (pu & ~qu) + (npv & ~nqv) - (pv & ~qv);
    }
    c.z += (~npu & nqu & 1u) - (~pu & qu & 1u) + (~npv & nqv & 1u) - (~pv & qv & 1u);
    c.w += npu - pu + npv - pv;
    if (valid) {
        ctr_store<CT>(cv.ctr, t, c);
        cv.fnow[t] = GROW ? step_cost_g(c.x, c.y, c.z, hbn, stepc[t], K) : step_cost(c.x, c.y, c.z, stepc[t], K);
    }
    uint32_t F = __ballot_sync(0xFFFFFFFFu, valid && c.w == cap);   // bit j <-> window bit j
    uint32_t V = __ballot_sync(0xFFFFFFFFu, valid);
    cv.own(u, lane);
    if (swap) cv.own(v, lane);
    if (lane < 2) {
        uint32_t M = ((1u << run) - 1u) << 1, NU = Nu, NV = Nv, sbit = s0 - 1;
        if (s0 == 0) { F >>= 1; V >>= 1; M >>= 1; NU >>= 1; NV >>= 1; sbit = 0; }
        const uint32_t wj = (sbit >> 5) + lane, sh = sbit & 31u;
        if (wj < S32 && (lane == 0 || sh != 0)) {
            // lane 0 holds the part of the window that falls into the first word, lane 1 the spill-over
            const uint32_t Vx = lane ? V >> (32 - sh) : V << sh, Fx = lane ? F >> (32 - sh) : F << sh;
            const uint32_t Mx = lane ? M >> (32 - sh) : M << sh;
            const uint32_t NUx = lane ? NU >> (32 - sh) : NU << sh, NVx = lane ? NV >> (32 - sh) : NV << sh;
            if (Vx) cv.full[wj] = (cv.full[wj] & ~Vx) | (Fx & Vx);
            if (Mx) {
                const size_t iu = (size_t)u * S32 + wj;
                cv.P[iu] = (cv.P[iu] & ~Mx) | (NUx & Mx);
                if (swap) {
                    const size_t iv = (size_t)v * S32 + wj;
                    cv.P[iv] = (cv.P[iv] & ~Mx) | (NVx & Mx);
                }
            }
        }
    }
    __syncwarp();
}

// PSMEM: the schedule lives in shared memory (16-bit counters); otherwise the chain's slice of global scratch is a
// copy-on-write overlay of the initial schedule (see kCowBitsMin).
// ASMEM (only with PSMEM): access bitmap and step constants staged in shared memory once per CTA.
// COLV (only without PSMEM): 2 or 4 when every column has exactly that many words, else 0 (see window_at).
template <bool PSMEM, bool GROW, bool ASMEM, int COLV>
__global__ void __launch_bounds__(PSMEM ? 256 : kWideGlobalThreads, 1)
wide_chain_kernel(const ChainParams prm)
{
    static_assert(PSMEM || !ASMEM, "shared access bitmap only beside shared schedules");
    static_assert(!PSMEM || COLV == 0, "vector columns only for schedules in global scratch");
    using CT = typename std::conditional<PSMEM, ushort4, uint4>::type;
    constexpr bool COW = !PSMEM;
    extern __shared__ uint4 smem4[];
    const uint32_t lane = threadIdx.x & 31, cic = threadIdx.x >> 5;
    const uint32_t cpb = blockDim.x >> 5;                         // chains per CTA
    const uint32_t slot = blockIdx.x * cpb + cic;
    const bool active = slot < prm.chain_count;
    const uint32_t chain = prm.chain_first + slot;
    const uint32_t S = prm.S, S32 = prm.S32, U = prm.U;
    const size_t pwords = (size_t)U * S32;
    const uint32_t c4 = PSMEM ? (S + 1) / 2 : S;                  // uint4 slots of the counters
    const uint32_t f4 = (S32 + 3) / 4, h4 = GROW ? (S + 3) / 4 : 0u;
    const uint32_t o4 = COW ? prm.cow_slots4 : 0u;
    const uint32_t fixed4 = wide_fixed4(S, S32, GROW, PSMEM, o4);
    uint4* const mine4 = smem4 + (size_t)cic * fixed4;
    WideView<CT, COW, COLV> cv;
    cv.ctr = reinterpret_cast<CT*>(mine4);
    cv.full = reinterpret_cast<uint32_t*>(mine4 + c4);
    cv.hb = reinterpret_cast<uint32_t*>(mine4 + c4 + f4);
    const uint32_t n4 = (S + 3) / 4;                              // uint4 slots of the present step costs
    cv.fnow = reinterpret_cast<uint32_t*>(mine4 + c4 + f4 + h4);
    cv.have = reinterpret_cast<uint32_t*>(mine4 + c4 + f4 + h4 + n4);
    WideScalars* const sc = reinterpret_cast<WideScalars*>(mine4 + c4 + f4 + h4 + n4 + o4);
    cv.win = mine4 + c4 + f4 + h4 + n4 + o4 + kWideScalars4;
    cv.acc = reinterpret_cast<int*>(cv.win + 2 * kWide);
    cv.nt = reinterpret_cast<uint8_t*>(cv.win + 2 * kWide + kWide / 4);
    cv.queue = reinterpret_cast<uint16_t*>(cv.win + 2 * kWide + kWide / 4 + kWide / 16);
    uint32_t* const pool = reinterpret_cast<uint32_t*>(smem4 + (size_t)cpb * fixed4);   // schedules, then A, then constants
    cv.P = PSMEM ? pool + (size_t)cic * pwords : prm.ws + (size_t)slot * pwords;
    cv.p0 = prm.Pcol0; cv.shift = prm.cow_shift; cv.U = U; cv.S32 = S32;
    const uint32_t* Acol = prm.Acol;
    const StepC* stepc = prm.stepc;
    if (ASMEM) {
        const size_t a_off = ((size_t)cpb * pwords + 3) & ~(size_t)3, c_off = (a_off + pwords + 3) & ~(size_t)3;
        uint32_t* const a_s = pool + a_off;
        StepC* const c_s = reinterpret_cast<StepC*>(pool + c_off);
        copy_words(a_s, prm.Acol, pwords, threadIdx.x, blockDim.x);
        for (uint32_t i = threadIdx.x; i < S; i += blockDim.x) c_s[i] = __ldg(prm.stepc + i);
        Acol = a_s;
        stepc = c_s;
    } else if (prm.stage_stepc) {                                 // the step constants alone, behind the chains' areas
        StepC* const c_s = reinterpret_cast<StepC*>(pool + (PSMEM ? (((size_t)cpb * pwords + 3) & ~(size_t)3) : 0));
        for (uint32_t i = threadIdx.x; i < S; i += blockDim.x) c_s[i] = __ldg(prm.stepc + i);
        stepc = c_s;
    }
    if (active) {
        for (uint32_t i = lane; i < S; i += 32) {
            const uint4 c0 = __ldg(prm.counters0 + i);
            const uint32_t hb0 = GROW ? __ldg(prm.hb0 + i) : 0u;
            ctr_store<CT>(cv.ctr, i, c0);
            if (GROW) cv.hb[i] = hb0;
            cv.fnow[i] = GROW ? step_cost_g(c0.x, c0.y, c0.z, hb0, __ldg(prm.stepc + i), prm.K)
                              : step_cost(c0.x, c0.y, c0.z, __ldg(prm.stepc + i), prm.K);
        }
        for (uint32_t i = lane; i < S32; i += 32) cv.full[i] = __ldg(prm.full0 + i);
        if (lane == 0) {
            sc->cur = sc->best = sc->best_at_boundary = prm.init_ticks;
            sc->best_move = ~0ull; sc->n_chg = 0; sc->hash = 0; sc->ulen = 0u; sc->snap_dirty = 0u; sc->qn = 0u;
            sc->n_again = sc->n_listed = sc->n_items = 0; sc->n_acc = sc->n_inf = 0;
        }
        if (COW) {
            for (uint32_t i = lane; i < prm.cow_slots4 * 4; i += 32) cv.have[i] = 0u;   // the slice holds nothing yet
        } else if (!(prm.state && prm.resume)) {
            copy_words_cold(cv.P, prm.Pcol0, pwords, lane);
        }
    }
    // the persistent part of a chain's shared memory: counters, full-step bitmap, written-to-HBM counts, present step
    // costs, overlay bitmap, scalars (everything before the per-batch work areas)
    const uint32_t persist4 = c4 + f4 + h4 + n4 + o4 + kWideScalars4;
    uint4* const saved = prm.state ? prm.state + (size_t)(chain - prm.hist_base) * prm.state4 : nullptr;
    if (active && saved && prm.resume) {
        __syncwarp();
        for (uint32_t i = lane; i < persist4; i += 32) mine4[i] = saved[i];
        if (PSMEM) copy_words_cold(cv.P, reinterpret_cast<const uint32_t*>(saved + persist4), pwords, lane);
    }
    __syncthreads();
    if (!active) return;
    uint32_t* snap = prm.snap ? prm.snap + (size_t)slot * pwords : nullptr;
    uint64_t* ulog = prm.undo_log ? prm.undo_log + (size_t)slot * prm.undo_cap : nullptr;

    uint64_t n_acc = 0, n_inf = 0;                                // per lane: of the proposals this lane owned

    // A segment of moves at one temperature: a level of the cooling schedule, or a round of a replica-exchange run.
    const bool exchange = prm.rung_hist != nullptr;
    uint64_t lvl_start = exchange ? (uint64_t)prm.round0 * prm.exch_every : 0;
    bool stop = false;
    for (uint32_t seg = exchange ? prm.round0 : 0u; seg < (exchange ? prm.round1 : prm.levels) && lvl_start < prm.upto; ++seg) {
        const uint32_t level = exchange ? prm.rung_hist[(size_t)seg * prm.hist_stride + (chain - prm.hist_base)] : seg;
        const uint64_t lvl_len = exchange ? min(prm.exch_every, prm.upto - lvl_start)
                                          : (level + 1 < prm.levels ? min(lvl_start + prm.per_level, prm.upto) : prm.upto) - lvl_start;
        const uint32_t shift = __ldg(prm.shifts + level);
        const uint32_t* trow = prm.table + (size_t)level * KVP_TABLE_Q;
        if (!exchange && level > 0) {
            const uint64_t best = sc->best, before = sc->best_at_boundary;
            if (prm.early_permille && level >= prm.early_from &&
                (before - best) * 1000ull < before * (uint64_t)prm.early_permille) {
                stop = true;
                break;
            }
            __syncwarp();
            if (lane == 0) sc->best_at_boundary = best;
            __syncwarp();
        }
        for (uint64_t off = 0; off < lvl_len; off += kWide) {
            const uint64_t m = lvl_start + off;
            const uint32_t nb = (uint32_t)min((uint64_t)kWide, lvl_len - off);
            WideMoves mv;
            mv.inf = mv.acc = mv.chg = 0u;
            uint32_t pend = 0u;                                   // bit h: this lane's row h is still to be committed
#pragma unroll
            for (int h = 0; h < kRows; ++h) {
                uint32_t r[4];
                const uint64_t mine = m + 32u * h + lane;
                philox4x32_10((uint32_t)mine, (uint32_t)(mine >> 32), chain, TAG_MOVE, prm.keys, r);
                LaneMove lm;
                decode_move(r, prm.p_swap_256, prm.len_choices, S, U, lm);
                mv.pk[h] = lm.pk; mv.u[h] = lm.u; mv.v[h] = lm.v; mv.w[h] = lm.w; mv.delta[h] = 0;
                if (32u * h + lane < nb) pend |= 1u << h;
            }
            uint32_t need = pend, stale = 0u;
            bool first_pass = true;
            // Evaluate what is named, then commit in move order as far as the evaluations are still good.
            for (;;) {
                wide_evaluate<GROW>(cv, Acol, prm.birth, stepc, prm.K, S, S32, trow, shift, need, first_pass, lane, mv, sc);
                first_pass = false;
                // Nearly always nothing in the batch changes the schedule: every lane counts its own proposals.
                if (!__any_sync(0xFFFFFFFFu, (mv.acc & mv.chg & ~mv.inf & pend) != 0u)) {
                    n_inf += __popc(mv.inf & pend);
                    n_acc += __popc(mv.acc & ~mv.inf & pend);
                    break;
                }
                bool stopped = false;
                for (uint32_t h = 0; h < kRows && !stopped; ++h) {
                    uint32_t rem = __ballot_sync(0xFFFFFFFFu, (pend >> h) & 1u);   // the row's lanes still to commit
                    if (!rem) continue;
                    const bool infl = (mv.inf >> h) & 1u, accl = !infl && ((mv.acc >> h) & 1u);
                    for (;;) {
                        const uint32_t st = __ballot_sync(0xFFFFFFFFu, (stale >> h) & 1u) & rem;
                        const uint32_t bl = __ballot_sync(0xFFFFFFFFu, accl && ((mv.chg >> h) & 1u)) & rem;
                        const uint32_t fst = st ? __ffs(st) - 1u : 32u, fbl = bl ? __ffs(bl) - 1u : 32u;
                        // the row's moves that are settled now: up to the next state-changing move (included), or up to
                        // the first proposal whose evaluation is stale (excluded), or all of them
                        const uint32_t upto_bit = fbl < fst ? fbl + 1u : fst;
                        const uint32_t done = upto_bit >= 32u ? rem : rem & ((1u << upto_bit) - 1u);
                        if ((done >> lane) & 1u) {
                            n_inf += infl ? 1u : 0u;
                            n_acc += accl ? 1u : 0u;
                            pend &= ~(1u << h);
                        }
                        rem &= ~done;
                        if (fbl < fst) {
                            // the next state-changing move, evaluated against the state as it is now: apply it
                            const uint32_t bb = fbl;
                            uint32_t pk = 0, bu = 0, bv = 0;
                            int delta = 0;
#pragma unroll
                            for (int k = 0; k < kRows; ++k)
                                if (h == (uint32_t)k) { pk = mv.pk[k]; bu = mv.u[k]; bv = mv.v[k]; delta = mv.delta[k]; }
                            pk = __shfl_sync(0xFFFFFFFFu, pk, bb); bu = __shfl_sync(0xFFFFFFFFu, bu, bb);
                            bv = __shfl_sync(0xFFFFFFFFu, bv, bb); delta = __shfl_sync(0xFFFFFFFFu, delta, bb);
                            const uint64_t after = (uint64_t)((int64_t)sc->cur + delta);
                            const bool leaving = snap && sc->snap_dirty && after >= sc->best;
                            if (leaving) copy_words(snap, cv.P, pwords, lane);   // leaving the best state: save it first
                            wide_apply<GROW>(cv, stepc, prm.K, S, S32, prm.cap, lane, h * 32 + bb, pk, bu, bv);
                            if (lane == 0) {
                                const uint64_t mb = m + 32u * h + bb;
                                if (leaving) sc->snap_dirty = 0u;
                                sc->cur = after;
                                ++sc->n_chg;
                                sc->hash = (sc->hash ^ mb) * 0x9E3779B97F4A7C15ull + after;
                                if (after < sc->best) { sc->best = after; sc->best_move = mb; sc->snap_dirty = 1u; sc->ulen = 0u; }
                                else if (ulog) {                          // every move is its own inverse: remember it
                                    const uint32_t ulen = sc->ulen;
                                    if (ulen < prm.undo_cap) ulog[ulen] = mb;
                                    if (ulen <= prm.undo_cap) sc->ulen = ulen + 1u;
                                }
                            }
                            __syncwarp();
                            // The applied move rewrote steps s0b .. s0b + len_b (bits, counters, full flags). A pending
                            // proposal read steps s0 - 1 .. s0 + len: its evaluation is stale iff the two ranges meet.
                            const uint32_t s0b = pk >> 8, endb = s0b + ((pk >> 1) & 63u);
#pragma unroll
                            for (int k = 0; k < kRows; ++k) {
                                const uint32_t s0 = mv.pk[k] >> 8, end = s0 + ((mv.pk[k] >> 1) & 63u);
                                if (s0 <= endb + 1 && s0b <= end) stale |= 1u << k;
                            }
                            stale &= pend;
                        } else if (fst < 32u) {
                            stopped = true;                       // a stale evaluation comes first
                            break;
                        } else {
                            break;                                // the row is done
                        }
                    }
                }
                if (!stopped) break;
                need = stale & pend;
                stale = 0u;
                const uint32_t again = __reduce_add_sync(0xFFFFFFFFu, __popc(need));
                if (lane == 0) sc->n_again += again;
            }
        }
        lvl_start += lvl_len;
    }
    const uint64_t m_end = stop || exchange ? lvl_start : prm.upto;   // moves done when the call ended
    // accepted and infeasible proposals were counted by the lanes that owned them
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        n_acc += __shfl_xor_sync(0xFFFFFFFFu, n_acc, off);
        n_inf += __shfl_xor_sync(0xFFFFFFFFu, n_inf, off);
    }
    n_acc += sc->n_acc; n_inf += sc->n_inf;                       // plus those of earlier calls on this state
    __syncwarp();
    if (lane == 0) { sc->n_acc = n_acc; sc->n_inf = n_inf; }
    __syncwarp();
    if (saved) {                                                  // the next round goes on from here
        for (uint32_t i = lane; i < persist4; i += 32) saved[i] = mine4[i];
        if (PSMEM) copy_words_cold(reinterpret_cast<uint32_t*>(saved + persist4), cv.P, pwords, lane);
    }
    if (snap && sc->snap_dirty) copy_words_cold(snap, cv.P, pwords, lane);
    if (ulog && lane == 0) prm.undo_len[slot] = sc->ulen;
    if (COW && prm.cow_out)                                       // which buckets the slice holds (for the walk back)
        for (uint32_t i = lane; i < prm.cow_slots4 * 4; i += 32)
            prm.cow_out[(size_t)slot * (prm.cow_slots4 * 4) + i] = cv.have[i];
    if (lane == 0) {
        kvp_chain_result res;
        res.best_ticks = sc->best; res.best_move = sc->best_move; res.final_ticks = sc->cur; res.moves_done = m_end;
        res.n_accepted = n_acc; res.n_changed = sc->n_chg; res.n_infeasible = n_inf; res.traj_hash = sc->hash;
        prm.results[chain - prm.result_base] = res;
        if (prm.work) {
            atomicAdd(prm.work, (unsigned long long)sc->n_again);
            atomicAdd(prm.work + 1, (unsigned long long)sc->n_listed);
            atomicAdd(prm.work + 2, (unsigned long long)sc->n_items);
        }
    }
    if (prm.dump && slot == 0) {
        __syncwarp();
        if (COW) copy_merged(prm.dump, cv.P, cv.p0, cv.have, cv.shift, U, S32, lane);
        else copy_words_cold(prm.dump, cv.P, pwords, lane);
    }
}

// Takes a finished chain's schedule back to its best state: the moves applied after the best were logged, each
// swap or flip is its own inverse, so applying them again in reverse order undoes them. One warp; only the
// schedule words are touched (the counters are not needed any more).
template <bool GROW>
__global__ void __launch_bounds__(32)
undo_kernel(const ChainParams prm, uint32_t slot)
{
    const uint32_t lane = threadIdx.x, S = prm.S, S32 = prm.S32;
    uint32_t* P = prm.ws + (size_t)slot * prm.U * S32;
    const uint64_t* ulog = prm.undo_log + (size_t)slot * prm.undo_cap;
    const uint32_t n = prm.undo_len[slot], chain = prm.chain_first + slot;
    for (uint32_t i = n; i-- > 0;) {
        const uint64_t m = ulog[i];
        uint32_t r[4];
        LaneMove mv;
        philox4x32_10((uint32_t)m, (uint32_t)(m >> 32), chain, TAG_MOVE, prm.keys, r);
        decode_move(r, prm.p_swap_256, prm.len_choices, S, prm.U, mv);
        const bool swap = mv.pk & 1u;
        const uint32_t len = (mv.pk >> 1) & 63u, s0 = mv.pk >> 8, end = min(s0 + len, S);
        if (lane < 2) {
            const uint32_t wj = (s0 >> 5) + lane;
            const uint32_t lo = max(s0, wj * 32u), hi = min(end, wj * 32u + 32u);
            if (hi > lo) {                               // run lengths are at most 30, so never a full word
                uint32_t mask = ((1u << (hi - lo)) - 1u) << (lo - wj * 32u);
                if (GROW) {                              // only the steps at which the units exist were touched
                    const uint32_t b = max(__ldg(prm.birth + mv.u), swap ? __ldg(prm.birth + mv.v) : 0u);
                    if (b >= wj * 32u + 32u) mask = 0u;
                    else if (b > wj * 32u) mask &= 0xFFFFFFFFu << (b - wj * 32u);
                }
                const size_t iu = (size_t)mv.u * S32 + wj, iv = (size_t)mv.v * S32 + wj;
                if (swap) {
                    const uint32_t a = P[iu], b = P[iv], d = (a ^ b) & mask;
                    if (d) { P[iu] = a ^ d; P[iv] = b ^ d; }
                } else {
                    P[iu] ^= mask;
                }
            }
        }
        __syncwarp();
    }
    // the schedule itself is copied out by gather_slice_kernel, on the whole GPU
}

// The schedule a slice of global scratch stands for, copied to dst: a plain slice (have == null) word for word; a
// copy-on-write slice bucket by bucket, from the slice where it holds the bucket and from the initial schedule
// elsewhere. A warp per bucket (per 1024 words of a plain slice).
__global__ void __launch_bounds__(256)
gather_slice_kernel(uint32_t* __restrict__ dst, const uint32_t* __restrict__ mine, const uint32_t* __restrict__ p0,
                    const uint32_t* __restrict__ have, uint32_t shift, uint32_t U, uint32_t S32)
{
    const uint32_t lane = threadIdx.x & 31, warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    if (have) {
        const uint32_t nb = (U + (1u << shift) - 1u) >> shift;
        for (uint32_t b = warp; b < nb; b += nwarps) {
            const size_t lo = (size_t)(b << shift) * S32, hi = (size_t)min(U, (b + 1u) << shift) * S32;
            const uint32_t* src = (have[b >> 5] >> (b & 31u)) & 1u ? mine : p0;
            for (size_t i = lo + lane; i < hi; i += 32) dst[i] = src[i];
        }
    } else {
        const size_t n = (size_t)U * S32;
        for (size_t lo = (size_t)warp * 1024; lo < n; lo += (size_t)nwarps * 1024)
            for (size_t i = lo + lane; i < min(n, lo + 1024); i += 32) dst[i] = mine[i];
    }
}

// bit t of full0 is set iff the initial schedule fills the HBM capacity at step t
__global__ void full_mask_kernel(const uint4* __restrict__ counters0, uint32_t S, uint32_t cap, uint32_t* __restrict__ full0)
{
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t bits = __ballot_sync(0xFFFFFFFFu, t < S && counters0[t < S ? t : 0].w == cap);
    if ((threadIdx.x & 31) == 0 && t < ((S + 31) / 32) * 32) full0[t >> 5] = bits;
}

// Calibration of the temperature ladder: proposals (i, 0, 0, TAG_CALIB), i < 1024, are evaluated against the
// initial schedule and never applied; acc = {sum of positive deltas, their number}.
template <bool GROW>
__global__ void __launch_bounds__(256)
calib_kernel(const ChainParams prm, unsigned long long* acc)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= CALIB_N) return;
    uint32_t r[4];
    LaneMove mv;
    philox4x32_10(i, 0u, 0u, TAG_CALIB, prm.keys, r);
    decode_move(r, prm.p_swap_256, prm.len_choices, prm.S, prm.U, mv);
    eval_lane<GROW>(prm.Pcol0, prm.Acol, prm.counters0, prm.full0, prm.birth, prm.hb0, prm.stepc, prm.K, prm.S, prm.S32,
                    prm.table, 0u, mv);
    if (!mv.inf && mv.delta > 0) {
        atomicAdd(acc, (unsigned long long)mv.delta);
        atomicAdd(acc + 1, 1ull);
    }
}

struct ReduceOut {
    uint64_t best_ticks, best_move, moves_total;
    uint32_t best_chain, pad;    // pad: the chains' error word
};

// Cross-chain best-so-far: lexicographic minimum of (best_ticks, chain index), plus the executed-move total.
__global__ void __launch_bounds__(1024)
reduce_kernel(const kvp_chain_result* __restrict__ res, uint32_t chains, const uint32_t* __restrict__ err, ReduceOut* out)
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
        out->pad = *err;                                  // a chain gave up waiting for its turn
    }
}

// One exchange round of a replica-exchange run: in every ladder the pairs of neighbouring rungs (j, j+1) with
// j = t (mod 2) may exchange. The chains keep their states; what changes hands is the rung, i.e. the temperature
// the chain runs at in the next round. A thread per ladder.
//   holder [ladders][rungs] : the chain (index within the call) that holds each rung; updated
//   rung_next [chains]      : the rungs for round t + 1 (the next row of the rung history)
//   counts                  : {exchanges tried, exchanges accepted}
struct ExchangeK {
    const kvp_chain_result* results;   // final_ticks = the chain's present cost
    uint32_t* holder;
    uint8_t* rung_next;
    uint32_t* n_exchanged;
    unsigned long long* counts;
    const uint32_t* xalways; const uint32_t* xtable; const uint32_t* xshifts;
    uint32_t ladders, rungs, first_ladder;
    uint32_t seed_lo, seed_hi;
    uint64_t t;
};

__global__ void __launch_bounds__(128)
exchange_kernel(const ExchangeK k)
{
    const uint32_t l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= k.ladders) return;
    uint32_t* hold = k.holder + (size_t)l * k.rungs;
    uint32_t tried = 0, done = 0;
    for (uint32_t j = (uint32_t)(k.t & 1ull); j + 1 < k.rungs; j += 2) {
        const uint32_t hot = hold[j], cold = hold[j + 1];
        const uint64_t Eh = k.results[hot].final_ticks, Ec = k.results[cold].final_ticks;
        bool accept;
        if (Eh <= Ec || k.xalways[j]) {
            accept = true;                                // the colder rung holds the worse schedule (or an equal one)
        } else {
            uint32_t x[4];
            philox4x32_10((uint32_t)k.t, (uint32_t)(k.t >> 32), (k.first_ladder + l) * k.rungs + j, TAG_EXCHANGE, k.seed_lo,
                          k.seed_hi, x);
            const uint64_t q = (Eh - Ec) >> k.xshifts[j];
            accept = q < KVP_TABLE_Q && x[3] < k.xtable[(size_t)j * KVP_TABLE_Q + q];
        }
        ++tried;
        if (accept) {
            hold[j] = cold; hold[j + 1] = hot;
            ++k.n_exchanged[hot]; ++k.n_exchanged[cold];
            ++done;
        }
    }
    for (uint32_t j = 0; j < k.rungs; ++j) k.rung_next[hold[j]] = (uint8_t)j;
    if (tried) {
        atomicAdd(k.counts, (unsigned long long)tried);
        atomicAdd(k.counts + 1, (unsigned long long)done);
    }
}

__global__ void exchange_init_kernel(uint32_t* holder, uint8_t* rung0, uint32_t* n_exchanged, uint32_t chains, uint32_t rungs)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= chains) return;
    holder[i] = i;                                        // chain i of the call starts on rung i % rungs of ladder i / rungs
    rung0[i] = (uint8_t)(i % rungs);
    n_exchanged[i] = 0u;
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
    uint32_t* full0;         // [S32]
    uint32_t* hb0;           // growing cache: [S] written-to-HBM counts of the initial schedule
    uint32_t* hb_tmp;        // growing cache: [S] the same for the winner's re-score
    bool grow;
    uint32_t* snap;          // best-state snapshots (shared-memory variant), or null
    uint64_t* undo_log;      // undo logs (global variant), or null
    uint32_t* undo_len;
    uint32_t undo_cap;
    uint32_t* cow_out;       // wide kernel, global variant: bucket bitmaps of the slices, or null
    uint32_t cow_shift;
    uint32_t cow_slots4;     // uint4 slots of a chain's bucket bitmap
    bool psmem;
    uint32_t wpb;            // chains per CTA
    uint32_t wpc;            // warps per chain
    uint32_t resident;       // chains per wave
    size_t smem_per_warp;    // shared memory per chain
    size_t smem_shared;      // shared memory of the CTA beside its chains (access bitmap and step constants)
    bool asmem;              // the access bitmap and the step constants are staged in shared memory
    bool wide;               // the wide kernel (one warp per chain, four proposals per lane)
    uint32_t S32;            // words per time-packed column
    bool stage_stepc;        // wide kernel: the step constants are staged in shared memory without the access bitmap
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
    if (a->moves / a->levels + a->levels >= (1ull << 36)) return KVP_ERR_RANGE;   // batches of a level are counted in 32 bits
    return KVP_OK;
}

typedef void (*ChainKernel)(const ChainParams);

template <bool PSMEM, bool ASMEM, bool COW>
ChainKernel chain_kernel_pick(bool grow, uint32_t W)
{
    if (W == 2) return grow ? chain_kernel<PSMEM, true, 2, ASMEM, COW> : chain_kernel<PSMEM, false, 2, ASMEM, COW>;
    return grow ? chain_kernel<PSMEM, true, 1, ASMEM, COW> : chain_kernel<PSMEM, false, 1, ASMEM, COW>;
}

ChainKernel chain_kernel_for(bool psmem, bool asmem, bool grow, uint32_t W, bool cow)
{
    if (!psmem) return cow ? chain_kernel_pick<false, false, true>(grow, W) : chain_kernel_pick<false, false, false>(grow, W);
    return asmem ? chain_kernel_pick<true, true, false>(grow, W) : chain_kernel_pick<true, false, false>(grow, W);
}

ChainKernel wide_kernel_for(bool psmem, bool asmem, bool grow, uint32_t S32)
{
    if (!psmem) {
        if (S32 == 2) return grow ? wide_chain_kernel<false, true, false, 2> : wide_chain_kernel<false, false, false, 2>;
        if (S32 == 4) return grow ? wide_chain_kernel<false, true, false, 4> : wide_chain_kernel<false, false, false, 4>;
        return grow ? wide_chain_kernel<false, true, false, 0> : wide_chain_kernel<false, false, false, 0>;
    }
    if (asmem) return grow ? wide_chain_kernel<true, true, true, 0> : wide_chain_kernel<true, false, true, 0>;
    return grow ? wide_chain_kernel<true, true, false, 0> : wide_chain_kernel<true, false, false, 0>;
}

ChainKernel kernel_of(const Ctx& c, bool psmem, bool asmem, uint32_t W)
{
    return c.wide ? wide_kernel_for(psmem, asmem, c.grow, c.S32) : chain_kernel_for(psmem, asmem, c.grow, W, c.cow_slots4 != 0);
}

int launch_chains(const Ctx& c, const ChainParams& prm, uint32_t count)
{
    const uint32_t grid = (count + c.wpb - 1) / c.wpb;
    const size_t smem = (size_t)c.wpb * c.smem_per_warp + c.smem_shared;
    kernel_of(c, c.psmem, c.asmem, c.wpc)<<<grid, c.wpb * c.wpc * 32, smem, c.st>>>(prm);
    KVP_CUDA(cudaGetLastError());
    return KVP_OK;
}

int run_chains(Ctx& c, uint32_t first, uint32_t count, uint32_t result_base, kvp_chain_result* results, uint64_t upto,
               uint32_t* dump, uint32_t* snap, bool with_undo = false)
{
    ChainParams prm = c.prm;
    prm.snap = snap;
    prm.undo_log = with_undo ? c.undo_log : nullptr; prm.undo_len = c.undo_len; prm.undo_cap = c.undo_cap;
    prm.cow_out = c.cow_out; prm.cow_shift = c.cow_shift; prm.cow_slots4 = c.cow_slots4;
    prm.stage_stepc = c.stage_stepc ? 1u : 0u;
    prm.chain_first = first; prm.chain_count = count; prm.result_base = result_base;
    prm.results = results; prm.upto = upto; prm.dump = dump;
    ++c.launches;
    return launch_chains(c, prm, count);
}

// Initial schedule, its counters and cost, the temperature ladder and the acceptance table.
int prepare(kvp_problem* p, const kvp_anneal_params* a, cudaStream_t st, Ctx& c, bool exchange = false)
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
    // per chain: counters, full-step bitmap and, per warp, the batch's windows, accumulators and work queue
    c.grow = p->dL != nullptr;
    const kvp_test_hooks hooks = g_hooks;
    c.S32 = p->S32;
    // Which kernel. Many chains per SM (more than 8, the jobs that fill the registers of an SM with one warp per
    // chain; more than 5 when the schedules fit shared memory): the wide kernel, which needs half the instructions
    // per proposal. Fewer chains per SM: the narrow kernel with two warps per chain, which hides the latency of a
    // chain's serial parts behind its second warp. A hot start (C_0 from p0 >= 0.5: a fifth of the proposals change
    // the schedule and the chain is a sequence of applied moves) on few chains: the narrow kernel with one warp per
    // chain, whose path through an applied move is the shortest.
    // kvp_set_test_hooks can force either (warps_per_chain 1 or 2: narrow; 3: wide).
    const uint32_t chains_per_sm = (a->chains + sms - 1) / sms;
    const size_t pbytes = (size_t)p->U * p->S32 * 4;
    const bool hot = !a->temps && a->p0 >= 0.5;
    const bool wide_in_smem = p->U < 65536u && (size_t)wide_fixed4(p->S, p->S32, c.grow, true, 0u) * 16 + pbytes <= budget / 2;
    c.wide = exchange || hooks.warps_per_chain == 3 ||
             (hooks.warps_per_chain == 0 && (chains_per_sm > 8 || (wide_in_smem && chains_per_sm > 5 && !hot)));
    // `shared`: the schedule is in shared memory (the wide kernel then keeps 16-bit counters)
    auto fixed_bytes = [&](uint32_t W, bool halfq = false, bool shared = true) {
        if (c.wide) return (size_t)wide_fixed4(p->S, p->S32, c.grow, shared, shared ? 0u : c.cow_slots4) * 16;
        return (size_t)chain_fixed4(p->S, p->S32, c.grow, W, halfq, shared ? 0u : c.cow_slots4) * 16;
    };
    c.stage_stepc = false;
    c.cow_slots4 = 0;
    c.cow_shift = 0;
    // Two warps per chain while that leaves an SM at most 16 warps (the registers allow no more): a job of few
    // chains then keeps twice as many warps in flight. kvp_set_test_hooks can override the choice (tests, tuning).
    uint32_t W = chains_per_sm <= 8 && !hot ? 2u : 1u;
    if (hooks.warps_per_chain == 1 || hooks.warps_per_chain == 2) W = hooks.warps_per_chain;
    if (c.wide) W = 1;
    c.psmem = fixed_bytes(1) + pbytes <= budget / 2 && (!c.wide || p->U < 65536u);
    if (c.psmem) {
        uint32_t want = chains_per_sm < 1 ? 1 : chains_per_sm;
        if (W == 2 && (want > 8 || (fixed_bytes(2) + pbytes) * want > budget) && (fixed_bytes(1) + pbytes) * want <= budget)
            W = 1;                                                 // the second warp's work area does not fit
        c.smem_per_warp = fixed_bytes(W) + pbytes;
        uint32_t wmax = (uint32_t)(budget / c.smem_per_warp);
        if (wmax > (c.wide ? 8u : 16u / W)) wmax = c.wide ? 8u : 16u / W;   // the wide kernel is built for CTAs of up to 256 threads
        c.wpb = want > wmax ? wmax : want;
        c.wpc = W;
        c.resident = a->chains;
        // the access bitmap and the step constants beside the schedules, if there is room (the offsets are the kernel's)
        const size_t a_off = ((size_t)c.wpb * (pbytes / 4) + 3) & ~(size_t)3, c_off = (a_off + pbytes / 4 + 3) & ~(size_t)3;
        const size_t with_a = (size_t)c.wpb * fixed_bytes(W, true) + c_off * 4 + (size_t)p->S * 16;
        c.asmem = with_a <= budget;
        if (c.asmem) {                                           // that kernel makes do with half the work queue
            c.smem_per_warp = fixed_bytes(W, true) + pbytes;
            c.smem_shared = with_a - (size_t)c.wpb * c.smem_per_warp;
        } else {
            c.smem_shared = 0;
            // the wide kernel stages at least the step constants when they fit
            const size_t with_c = (size_t)c.wpb * c.smem_per_warp + 16 + (size_t)p->S * 16;
            if (c.wide && with_c <= budget) {
                c.stage_stepc = true;
                c.smem_shared = with_c - (size_t)c.wpb * c.smem_per_warp;
            }
        }
        KVP_CUDA(cudaFuncSetAttribute(kernel_of(c, true, c.asmem, W), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)budget));
    } else {
        {
            // Copy-on-write slices: always for the wide kernel; for the narrow kernel where whole copies of the initial
            // schedule would add up to gigabytes (growing_8b: 1024 x 17 MB, a third of the kernel's time), not where
            // they are small (layer_8b: 1024 x 512 KB), because a take-over lengthens the path through an applied move
            // (layer_8b 14.0 -> 16.0 ms with it).
            const size_t per_sm_max = c.wide ? kWideGlobalThreads / 32 : 16 / W;
            const size_t most = a->chains < per_sm_max * sms ? a->chains : per_sm_max * sms;
            const bool overlay = c.wide || (hooks.overlay ? hooks.overlay == 1 : most * col_bytes >= ((size_t)4 << 30));
            c.cow_slots4 = 0;
            c.cow_shift = 0;
            if (overlay) {
                // The bucket bitmap takes what a full CTA of chains leaves of the shared memory: the smaller the
                // buckets, the fewer reads of a long chain go to its private slice.
                const size_t bare = fixed_bytes(W, false, false);
                const size_t stepc_bytes = c.wide && (size_t)p->S * 16 <= 32768 ? (size_t)p->S * 16 : 0;
                uint32_t per_cta = c.wide ? kWideGlobalThreads / 32 : 16 / W;     // chains of a full CTA
                if (chains_per_sm < per_cta) per_cta = chains_per_sm ? chains_per_sm : 1u;
                if ((budget - stepc_bytes) / bare < per_cta) per_cta = (uint32_t)((budget - stepc_bytes) / bare);
                if (per_cta < 1) return KVP_ERR_RANGE;
                const size_t share = (budget - stepc_bytes) / per_cta;
                size_t bits = share > bare ? (share - bare) / 16 * 128 : 0;
                if (bits < kCowBitsMin) bits = kCowBitsMin;
                if (bits > kCowBitsMax) bits = kCowBitsMax;
                c.cow_shift = 0;
                while (((uint64_t)p->U + (1ull << c.cow_shift) - 1) >> c.cow_shift > bits) ++c.cow_shift;
                const uint64_t buckets = ((uint64_t)p->U + (1ull << c.cow_shift) - 1) >> c.cow_shift;
                c.cow_slots4 = (uint32_t)((buckets + 127) / 128);
            }
            const size_t ctr_bytes = fixed_bytes(W, false, false);
            if (ctr_bytes > budget) return KVP_ERR_RANGE;
            c.smem_per_warp = ctr_bytes;
            c.smem_shared = 0;
            c.asmem = false;
            c.wpc = W;
            // the wide kernel stages the step constants once per CTA when they are small
            c.stage_stepc = c.wide && (size_t)p->S * 16 <= 32768 && ctr_bytes + (size_t)p->S * 16 <= budget;
            if (c.stage_stepc) c.smem_shared = (size_t)p->S * 16;
            uint32_t wcap = (uint32_t)((budget - c.smem_shared) / ctr_bytes);   // chains per CTA at most
            if (wcap > 16 / W) wcap = 16 / W;
            if (c.wide && wcap > kWideGlobalThreads / 32) wcap = kWideGlobalThreads / 32;
            KVP_CUDA(cudaFuncSetAttribute(kernel_of(c, false, false, W), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)budget));
            int ctas = 0;
            KVP_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&ctas, kernel_of(c, false, false, W), (int)(wcap * W * 32),
                                                                   wcap * c.smem_per_warp + c.smem_shared));
            if (ctas < 1) return KVP_ERR_RANGE;
            uint32_t per_sm = (uint32_t)ctas * wcap;                   // resident chains per SM, at most 32 warps
            if (per_sm * W > 32) per_sm = 32 / W / wcap ? 32 / W / wcap * wcap : wcap;
            size_t free_b = 0, total_b = 0;
            KVP_CUDA(cudaMemGetInfo(&free_b, &total_b));
            free_b += p->chain_ws_bytes;                               // what we already hold can be reused
            {                                                          // and so can what the pool holds in reserve
                cudaMemPool_t pool; uint64_t reserved = 0, used = 0;
                if (cudaDeviceGetDefaultMemPool(&pool, dev) == cudaSuccess &&
                    cudaMemPoolGetAttribute(pool, cudaMemPoolAttrReservedMemCurrent, &reserved) == cudaSuccess &&
                    cudaMemPoolGetAttribute(pool, cudaMemPoolAttrUsedMemCurrent, &used) == cudaSuccess && reserved > used)
                    free_b += (size_t)(reserved - used);
            }
            const size_t usable = free_b / 10 * 7;
            size_t fit = usable / col_bytes;
            if (fit < 1) return KVP_ERR_NOMEM;
            size_t cap_r = (size_t)per_sm * sms;
            size_t r = a->chains < cap_r ? a->chains : cap_r;
            if (r > fit) r = fit;
            // test hook: at most n chains at a time, so that small jobs come in several waves
            if (hooks.resident >= 1 && (size_t)hooks.resident < r) r = hooks.resident;
            const uint32_t waves = (uint32_t)((a->chains + r - 1) / r);
            c.resident = (a->chains + waves - 1) / waves;              // equal waves
            // a wave is spread over all SMs: CTAs of ceil(resident / SMs) chains where one CTA per SM holds them
            const uint32_t even = (c.resident + sms - 1) / sms;
            c.wpb = even < wcap ? even : wcap;
        }
    }
    // a replica-exchange run keeps every chain's slice between its rounds: all chains have to be resident at once
    if (exchange && !c.psmem && a->chains > c.resident) return KVP_ERR_RANGE;

    // workspace layout
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += align256(bytes); return o; };
    const size_t o_P0 = take(sched_bytes), o_col0 = take(col_bytes), o_cnt = take((size_t)p->S * 16);
    const size_t o_small = take(256), o_table = take((size_t)a->levels * KVP_TABLE_Q * 4), o_shift = take((size_t)a->levels * 4);
    const size_t o_res = take((size_t)(a->chains + 1) * sizeof(kvp_chain_result));
    const size_t o_dump = take(col_bytes), o_sched = take(sched_bytes);
    const size_t o_slots = take(c.psmem ? 0 : (size_t)c.resident * col_bytes);
    const size_t o_full = take((size_t)p->S32 * 4);
    const size_t o_hb0 = take(c.grow ? (size_t)p->S * 4 : 0), o_hbt = take(c.grow ? (size_t)p->S * 4 : 0);
    // Chains whose schedule lives in shared memory save it to global memory whenever they leave their best state;
    // chains in global scratch do not (a copy would cost as much as thousands of moves): their winner is replayed.
    const size_t snap_bytes = (size_t)a->chains * p->U * p->S32 * 4;
    const bool snapshots = c.psmem && snap_bytes <= ((size_t)2 << 30);
    const size_t o_snap = take(snapshots ? snap_bytes : 0);
    // Chains in global scratch log the moves they apply after their best state (8 bytes each, up to 4096), so that
    // the winner can be walked back instead of replayed from its first move.
    c.undo_cap = c.psmem ? 0u : 4096u;
    const size_t o_ulog = take((size_t)c.resident * c.undo_cap * 8), o_ulen = take(c.psmem ? 0 : (size_t)c.resident * 4);
    // Where the chains come in several waves they also log the units they rewrite (4 bytes each, up to 16384): the
    // chain that takes over the slice in the next wave copies only those from the initial schedule again, not all of it.
    const bool cow = !c.psmem && c.cow_slots4 != 0;
    const size_t o_cow = take(cow ? (size_t)c.resident * c.cow_slots4 * 16 : 0);
    rc = ensure_chain_ws(p, off, st);
    if (rc) return rc;
    char* base = static_cast<char*>(p->d_chain_ws);
    c.P0 = (uint32_t*)(base + o_P0); c.Pcol0 = (uint32_t*)(base + o_col0); c.counts0 = (uint32_t*)(base + o_cnt);
    c.small = (uint64_t*)(base + o_small); c.table = (uint32_t*)(base + o_table); c.shifts = (uint32_t*)(base + o_shift);
    c.results = (kvp_chain_result*)(base + o_res); c.dumpcol = (uint32_t*)(base + o_dump);
    c.sched = (uint32_t*)(base + o_sched); c.slots = (uint32_t*)(base + o_slots);
    c.hb0 = c.grow ? (uint32_t*)(base + o_hb0) : nullptr; c.hb_tmp = c.grow ? (uint32_t*)(base + o_hbt) : nullptr;
    c.full0 = (uint32_t*)(base + o_full); c.snap = snapshots ? (uint32_t*)(base + o_snap) : nullptr;
    c.undo_log = c.psmem ? nullptr : (uint64_t*)(base + o_ulog); c.undo_len = c.psmem ? nullptr : (uint32_t*)(base + o_ulen);
    c.cow_out = cow ? (uint32_t*)(base + o_cow) : nullptr;

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
        if (!c.grow && (rc = launch_row_to_columns(row, p->U, p->S, p->S32, c.Pcol0, st))) return rc;
        c.launches += 2;
    }
    if (c.grow) {
        // a unit of the initial placement enters HBM when it is written; the chains keep the bits before that clear
        if ((rc = launch_and_rows(c.P0, p->dL, (size_t)p->S * p->W32, st))) return rc;
        if ((rc = launch_bit_transpose(c.P0, p->S, p->W32, p->U, c.Pcol0, p->S32, st))) return rc;
        c.launches += a->init_mode == KVP_INIT_USER ? 2 : 1;
    }
    if ((rc = launch_counts(p, c.P0, 1, c.counts0, c.hb0, st, &c.launches))) return rc;
    if ((rc = launch_finish(p, c.counts0, c.hb0, 1, nullptr, c.small, nullptr, nullptr, (int32_t*)(c.small + 2), c.small + 1,
                            st)))
        return rc;
    ++c.launches;
    full_mask_kernel<<<(p->S32 * 32 + 255) / 256, 256, 0, st>>>((const uint4*)c.counts0, p->S, p->cap, c.full0);
    KVP_CUDA(cudaGetLastError());
    ++c.launches;

    ChainParams& prm = c.prm;
    memset(&prm, 0, sizeof prm);
    prm.Acol = p->dAcol; prm.stepc = p->d_stepc; prm.counters0 = (const uint4*)c.counts0; prm.Pcol0 = c.Pcol0;
    prm.table = c.table; prm.shifts = c.shifts; prm.ws = c.slots; prm.K = p->K; prm.full0 = c.full0;
    prm.birth = p->d_birth; prm.hb0 = c.hb0;
    prm.err = reinterpret_cast<uint32_t*>(c.small + 16);
    prm.work = nullptr;                                   // set by kvp_anneal for the chains of the search proper
    // test hook (tests of the bounded wait only): one hand-over per chain is withheld, the waiting warp gives up
    // after its poll limit (about a second) and the call returns KVP_ERR_TIMEOUT
    prm.drop_first_turn = hooks.drop_turn ? 1u : 0u;
    // test hook: batches with more than n < 496 queue items already take the two-halves path of the half-size work
    // queue, which ordinary inputs almost never reach
    prm.split_at = kQueueCap / 2;
    if (hooks.split_queue_plus1 >= 1 && hooks.split_queue_plus1 - 1 < kQueueCap / 2) prm.split_at = hooks.split_queue_plus1 - 1;
    KVP_CUDA(cudaMemsetAsync(prm.err, 0, 4, st));
    prm.U = p->U; prm.S = p->S; prm.S32 = p->S32; prm.cap = p->cap;
    prm.levels = a->levels; prm.p_swap_256 = a->p_swap_256; prm.len_choices = a->max_len_log2 + 1;
    prm.early_permille = a->early_stop_permille; prm.early_from = a->early_stop_from_level;
    prm.keys = philox_keys((uint32_t)a->seed, (uint32_t)(a->seed >> 32));
    prm.per_level = a->moves / a->levels ? a->moves / a->levels : 1;

    // temperature ladder
    c.temps.resize(a->levels);
    c.calib_mean = 0;
    const bool calibrate = a->temps == nullptr;
    if (calibrate) {
        KVP_CUDA(cudaMemsetAsync(c.small + 4, 0, 16, st));
        if (c.grow) calib_kernel<true><<<CALIB_N / 256, 256, 0, st>>>(prm, (unsigned long long*)(c.small + 4));
        else calib_kernel<false><<<CALIB_N / 256, 256, 0, st>>>(prm, (unsigned long long*)(c.small + 4));
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
    if ((rc = run_chains(c, chain, 1, chain, result_dev, upto, c.dumpcol, nullptr))) return rc;
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
    struct Events {                                       // destroyed on every way out of the call
        cudaEvent_t e[4];
        int n = 0;
        ~Events() { for (int i = 0; i < n; ++i) cudaEventDestroy(e[i]); }
        cudaEvent_t operator[](int i) const { return e[i]; }
    } ev;
    for (; ev.n < 4; ++ev.n) KVP_CUDA(cudaEventCreate(&ev.e[ev.n]));
    KVP_CUDA(cudaEventRecord(ev[0], st));
    if ((rc = prepare(p, a, st, c))) return rc;
    KVP_CUDA(cudaEventRecord(ev[1], st));

    // the chains, one wave of resident chains after the other
    ReduceOut* red_dev = reinterpret_cast<ReduceOut*>(c.small + 8);
    ReduceOut red;
    memset(&red, 0, sizeof red);
    uint32_t dumped_chain = 0xFFFFFFFFu;                  // call-local index of the chain whose best state is in dumpcol
    uint32_t waves = 0;
    unsigned long long* work_dev = reinterpret_cast<unsigned long long*>(c.small + 24);
    KVP_CUDA(cudaMemsetAsync(work_dev, 0, 24, st));
    c.prm.work = c.wide ? work_dev : nullptr;
    for (uint32_t first = 0; first < a->chains; first += c.resident, ++waves) {
        const uint32_t count = a->chains - first < c.resident ? a->chains - first : c.resident;
        if ((rc = run_chains(c, a->first_chain + first, count, a->first_chain, c.results, a->moves, nullptr, c.snap,
                             c.undo_log != nullptr)))
            return rc;
        if (c.undo_log) {
            // Best so far over the chains that have finished; if it belongs to this wave, walk that chain back to
            // its best state while its scratch slice still holds its final state.
            reduce_kernel<<<1, 1024, 0, st>>>(c.results, first + count, c.prm.err, red_dev);
            KVP_CUDA(cudaGetLastError());
            ++c.launches;
            KVP_CUDA(cudaMemcpyAsync(&red, red_dev, sizeof red, cudaMemcpyDeviceToHost, st));
            KVP_CUDA(cudaStreamSynchronize(st));
            if (red.pad) return KVP_ERR_TIMEOUT;
            if (red.best_chain >= first && red.best_move != ~0ull) {
                uint32_t len = 0;
                KVP_CUDA(cudaMemcpyAsync(&len, c.undo_len + (red.best_chain - first), 4, cudaMemcpyDeviceToHost, st));
                KVP_CUDA(cudaStreamSynchronize(st));
                if (len <= c.undo_cap) {
                    ChainParams prm = c.prm;
                    prm.chain_first = a->first_chain + first;
                    prm.undo_log = c.undo_log; prm.undo_len = c.undo_len; prm.undo_cap = c.undo_cap;
                    prm.cow_out = c.cow_out; prm.cow_shift = c.cow_shift; prm.cow_slots4 = c.cow_slots4;
                    const uint32_t wslot = red.best_chain - first;
                    if (c.grow) undo_kernel<true><<<1, 32, 0, st>>>(prm, wslot);
                    else undo_kernel<false><<<1, 32, 0, st>>>(prm, wslot);
                    KVP_CUDA(cudaGetLastError());
                    gather_slice_kernel<<<148 * 4, 256, 0, st>>>(c.dumpcol, c.slots + (size_t)wslot * p->U * p->S32, c.Pcol0,
                                                                 c.cow_out ? c.cow_out + (size_t)wslot * (c.cow_slots4 * 4) : nullptr,
                                                                 c.cow_shift, p->U, p->S32);
                    KVP_CUDA(cudaGetLastError());
                    c.launches += 2;
                    dumped_chain = red.best_chain;
                }
            }
        }
    }
    KVP_CUDA(cudaEventRecord(ev[2], st));
    c.prm.work = nullptr;                                 // a replay of the winner is not part of the count
    unsigned long long work[3] = {0, 0, 0};
    KVP_CUDA(cudaMemcpyAsync(work, work_dev, sizeof work, cudaMemcpyDeviceToHost, st));

    // cross-chain reduction, then the winner's schedule (its own snapshot, its walked-back state, or a replay) and a
    // re-score
    if (!c.undo_log) {
        reduce_kernel<<<1, 1024, 0, st>>>(c.results, a->chains, c.prm.err, red_dev);
        KVP_CUDA(cudaGetLastError());
        ++c.launches;
        KVP_CUDA(cudaMemcpyAsync(&red, red_dev, sizeof red, cudaMemcpyDeviceToHost, st));
        KVP_CUDA(cudaStreamSynchronize(st));
        if (red.pad) return KVP_ERR_TIMEOUT;
    }
    const uint64_t upto = red.best_move == ~0ull ? 0 : red.best_move + 1;
    if (upto && (c.snap || dumped_chain == red.best_chain)) {
        const uint32_t* col = c.snap ? c.snap + (size_t)red.best_chain * p->U * p->S32 : c.dumpcol;
        if ((rc = launch_bit_transpose(col, p->U, p->S32, p->S, c.sched, p->W32, st))) return rc;
        ++c.launches;
        red.best_chain += a->first_chain;                  // the reduction works on call-local indices
    } else {
        red.best_chain += a->first_chain;
        if ((rc = replay_to_sched(p, c, red.best_chain, upto, c.results + a->chains))) return rc;
    }
    if ((rc = launch_counts(p, c.sched, 1, c.counts0, c.hb_tmp, st, &c.launches))) return rc;
    if ((rc = launch_finish(p, c.counts0, c.hb_tmp, 1, nullptr, c.small, nullptr, nullptr, (int32_t*)(c.small + 2),
                            c.small + 1, st)))
        return rc;
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
        stats->chain_launches = waves; stats->resident_chains = c.resident;
        stats->wide_kernel = c.wide ? 1u : 0u;
        stats->work_again = work[0]; stats->work_listed = work[1]; stats->work_items = work[2];
    }
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
    uint32_t gave_up = 0;
    KVP_CUDA(cudaMemcpyAsync(&gave_up, c.prm.err, 4, cudaMemcpyDeviceToHost, st));
    KVP_CUDA(cudaStreamSynchronize(st));
    return gave_up ? KVP_ERR_TIMEOUT : KVP_OK;
}

extern "C" void kvp_set_test_hooks(const kvp_test_hooks* hooks)
{
    if (hooks) g_hooks = *hooks;
    else memset(&g_hooks, 0, sizeof g_hooks);
}

extern "C" int kvp_exchange_temps(const double* temps, uint32_t rungs, double* pair_temps, uint32_t* always)
{
    if (!temps || !rungs || (rungs > 1 && (!pair_temps || !always))) return KVP_ERR_ARG;
    for (uint32_t j = 0; j + 1 < rungs; ++j) {
        const double a = temps[j] >= 1.0 ? temps[j] : 1.0, b = temps[j + 1] >= 1.0 ? temps[j + 1] : 1.0;
        if (b > a) return KVP_ERR_ARG;                     // a ladder falls
        const double inv = 1.0 / b - 1.0 / a;
        if (!(inv > 0.0) || 1.0 / inv > 1099511627776.0) { always[j] = 1; pair_temps[j] = 1.0; }
        else { always[j] = 0; pair_temps[j] = 1.0 / inv; }
    }
    return KVP_OK;
}

extern "C" int kvp_anneal_exchange(kvp_problem* p, const kvp_anneal_params* a, const kvp_exchange_params* xp,
                                   uint32_t* best_schedule, uint64_t* best_ticks, double* best_seconds,
                                   kvp_anneal_stats* stats, uint32_t* final_rung, uint32_t* n_exchanged, void* stream)
{
    Ctx c;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc = validate(p, a);
    if (rc) return rc;
    if (!xp || !xp->rungs || xp->rungs > 256 || xp->reserved || !xp->exchange_every) return KVP_ERR_ARG;
    const uint32_t rungs = xp->rungs, chains = a->chains;
    if (a->levels != rungs || chains % rungs || a->first_chain % rungs || a->early_stop_permille) return KVP_ERR_ARG;
    const uint64_t rounds64 = (a->moves + xp->exchange_every - 1) / xp->exchange_every;
    if (rounds64 * chains > (1ull << 30)) return KVP_ERR_RANGE;          // the rung history is kept: one byte per chain and round
    const uint32_t rounds = (uint32_t)rounds64;
    KVP_CUDA(cudaSetDevice(p->device));
    struct Events {
        cudaEvent_t e[4];
        int n = 0;
        ~Events() { for (int i = 0; i < n; ++i) cudaEventDestroy(e[i]); }
        cudaEvent_t operator[](int i) const { return e[i]; }
    } ev;
    for (; ev.n < 4; ++ev.n) KVP_CUDA(cudaEventCreate(&ev.e[ev.n]));
    KVP_CUDA(cudaEventRecord(ev[0], st));
    if ((rc = prepare(p, a, st, c, true))) return rc;

    // exchange thresholds of the pairs of neighbouring rungs: the move table's form at the pair temperatures
    const uint32_t pairs = rungs > 1 ? rungs - 1 : 1;
    std::vector<double> pair_temps(pairs, 1.0);
    std::vector<uint32_t> always(pairs, 0u), xtable((size_t)pairs * KVP_TABLE_Q), xshifts(pairs);
    if ((rc = kvp_exchange_temps(c.temps.data(), rungs, pair_temps.data(), always.data()))) return rc;
    if ((rc = kvp_accept_table(pair_temps.data(), pairs, xtable.data(), xshifts.data()))) return rc;

    // workspace of the run: rung history, holders, exchange counts, thresholds, the chains' saved states
    const uint32_t persist4 = wide_persist4(p->S, p->S32, c.grow, c.psmem, c.cow_slots4);
    const size_t pwords = (size_t)p->U * p->S32;
    const uint32_t state4 = persist4 + (c.psmem ? (uint32_t)((pwords + 3) / 4) : 0u);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += align256(bytes); return o; };
    const size_t o_hist = take((size_t)rounds * chains), o_hold = take((size_t)chains * 4), o_nex = take((size_t)chains * 4);
    const size_t o_cnt = take(16), o_alw = take((size_t)pairs * 4), o_xsh = take((size_t)pairs * 4);
    const size_t o_xt = take((size_t)pairs * KVP_TABLE_Q * 4), o_state = take((size_t)chains * state4 * 16);
    char* xw = nullptr;
    KVP_CUDA(cudaMallocAsync(&xw, off, st));
    struct Free {                                          // in stream order, on every way out
        char* ptr; cudaStream_t st;
        ~Free() { cudaFreeAsync(ptr, st); }
    } guard{xw, st};
    uint8_t* hist = (uint8_t*)(xw + o_hist);
    uint32_t* holder = (uint32_t*)(xw + o_hold);
    uint32_t* nex = (uint32_t*)(xw + o_nex);
    unsigned long long* counts = (unsigned long long*)(xw + o_cnt);
    KVP_CUDA(cudaMemsetAsync(counts, 0, 16, st));
    KVP_CUDA(cudaMemcpyAsync(xw + o_alw, always.data(), (size_t)pairs * 4, cudaMemcpyHostToDevice, st));
    KVP_CUDA(cudaMemcpyAsync(xw + o_xsh, xshifts.data(), (size_t)pairs * 4, cudaMemcpyHostToDevice, st));
    KVP_CUDA(cudaMemcpyAsync(xw + o_xt, xtable.data(), xtable.size() * 4, cudaMemcpyHostToDevice, st));
    exchange_init_kernel<<<(chains + 255) / 256, 256, 0, st>>>(holder, hist, nex, chains, rungs);
    KVP_CUDA(cudaGetLastError());
    ++c.launches;
    KVP_CUDA(cudaEventRecord(ev[1], st));

    ChainParams prm = c.prm;
    prm.snap = c.snap; prm.undo_log = nullptr;
    prm.cow_out = nullptr; prm.cow_shift = c.cow_shift; prm.cow_slots4 = c.cow_slots4;
    prm.stage_stepc = c.stage_stepc ? 1u : 0u;
    prm.chain_first = a->first_chain; prm.chain_count = chains; prm.result_base = a->first_chain;
    prm.results = c.results; prm.upto = a->moves; prm.dump = nullptr;
    prm.rung_hist = hist; prm.exch_every = xp->exchange_every; prm.hist_stride = chains; prm.hist_base = a->first_chain;
    prm.state = (uint4*)(xw + o_state); prm.state4 = state4;
    unsigned long long* work_dev = reinterpret_cast<unsigned long long*>(c.small + 24);
    KVP_CUDA(cudaMemsetAsync(work_dev, 0, 24, st));
    ExchangeK xk;
    xk.results = c.results; xk.holder = holder; xk.n_exchanged = nex; xk.counts = counts;
    xk.xalways = (const uint32_t*)(xw + o_alw); xk.xtable = (const uint32_t*)(xw + o_xt); xk.xshifts = (const uint32_t*)(xw + o_xsh);
    xk.ladders = chains / rungs; xk.rungs = rungs; xk.first_ladder = a->first_chain / rungs;
    xk.seed_lo = (uint32_t)a->seed; xk.seed_hi = (uint32_t)(a->seed >> 32);
    for (uint32_t t = 0; t < rounds; ++t) {
        prm.round0 = t; prm.round1 = t + 1; prm.resume = t > 0 ? 1u : 0u;
        prm.work = t + 1 == rounds ? work_dev : nullptr;   // the counts travel with the saved state; the last round reports
        if ((rc = launch_chains(c, prm, chains))) return rc;
        ++c.launches;
        if (t + 1 < rounds) {
            xk.t = t; xk.rung_next = hist + (size_t)(t + 1) * chains;
            exchange_kernel<<<(xk.ladders + 127) / 128, 128, 0, st>>>(xk);
            KVP_CUDA(cudaGetLastError());
            ++c.launches;
        }
    }
    KVP_CUDA(cudaEventRecord(ev[2], st));

    ReduceOut* red_dev = reinterpret_cast<ReduceOut*>(c.small + 8);
    ReduceOut red;
    reduce_kernel<<<1, 1024, 0, st>>>(c.results, chains, c.prm.err, red_dev);
    KVP_CUDA(cudaGetLastError());
    ++c.launches;
    unsigned long long work[3] = {0, 0, 0}, xcounts[2] = {0, 0};
    KVP_CUDA(cudaMemcpyAsync(&red, red_dev, sizeof red, cudaMemcpyDeviceToHost, st));
    KVP_CUDA(cudaMemcpyAsync(work, work_dev, sizeof work, cudaMemcpyDeviceToHost, st));
    KVP_CUDA(cudaMemcpyAsync(xcounts, counts, sizeof xcounts, cudaMemcpyDeviceToHost, st));
    KVP_CUDA(cudaStreamSynchronize(st));
    // the winner's schedule: its snapshot, or a replay of that one chain through the rungs it held
    const uint64_t upto = red.best_move == ~0ull ? 0 : red.best_move + 1;
    if (upto == 0) {
        KVP_CUDA(cudaMemcpyAsync(c.sched, c.P0, (size_t)p->S * p->W32 * 4, cudaMemcpyDeviceToDevice, st));
    } else if (c.snap) {
        if ((rc = launch_bit_transpose(c.snap + (size_t)red.best_chain * pwords, p->U, p->S32, p->S, c.sched, p->W32, st))) return rc;
        ++c.launches;
    } else {
        ChainParams rp = prm;
        rp.snap = nullptr; rp.state = nullptr; rp.resume = 0u; rp.work = nullptr;
        rp.chain_first = a->first_chain + red.best_chain; rp.chain_count = 1; rp.result_base = rp.chain_first;
        rp.results = c.results + chains; rp.upto = upto; rp.dump = c.dumpcol;
        rp.round0 = 0; rp.round1 = rounds;
        if ((rc = launch_chains(c, rp, 1))) return rc;
        if ((rc = launch_bit_transpose(c.dumpcol, p->U, p->S32, p->S, c.sched, p->W32, st))) return rc;
        c.launches += 2;
    }
    red.best_chain += a->first_chain;
    if ((rc = launch_counts(p, c.sched, 1, c.counts0, c.hb_tmp, st, &c.launches))) return rc;
    if ((rc = launch_finish(p, c.counts0, c.hb_tmp, 1, nullptr, c.small, nullptr, nullptr, (int32_t*)(c.small + 2),
                            c.small + 1, st)))
        return rc;
    ++c.launches;
    if (best_schedule)
        KVP_CUDA(cudaMemcpyAsync(best_schedule, c.sched, (size_t)p->S * p->W32 * 4, cudaMemcpyDeviceToDevice, st));
    uint64_t host_small[4];
    KVP_CUDA(cudaMemcpyAsync(host_small, c.small, sizeof host_small, cudaMemcpyDeviceToHost, st));
    if (stats && stats->per_chain)
        KVP_CUDA(cudaMemcpyAsync(stats->per_chain, c.results, (size_t)chains * sizeof(kvp_chain_result), cudaMemcpyDeviceToHost, st));
    std::vector<uint8_t> last_row(final_rung ? chains : 0);
    if (final_rung)
        KVP_CUDA(cudaMemcpyAsync(last_row.data(), hist + (size_t)(rounds - 1) * chains, chains, cudaMemcpyDeviceToHost, st));
    if (n_exchanged) KVP_CUDA(cudaMemcpyAsync(n_exchanged, nex, (size_t)chains * 4, cudaMemcpyDeviceToHost, st));
    KVP_CUDA(cudaEventRecord(ev[3], st));
    KVP_CUDA(cudaStreamSynchronize(st));
    if (final_rung)
        for (uint32_t i = 0; i < chains; ++i) final_rung[i] = last_row[i];
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
        stats->chain_launches = rounds; stats->resident_chains = chains; stats->wide_kernel = 1u;
        stats->work_again = work[0]; stats->work_listed = work[1]; stats->work_items = work[2];
        stats->exchange_rounds = rounds; stats->exchanges_tried = xcounts[0]; stats->exchanges_accepted = xcounts[1];
    }
    return ok ? KVP_OK : KVP_ERR_INTERNAL;
}
