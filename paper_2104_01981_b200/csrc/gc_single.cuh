// Exact top-k of ONE large tensor in one cooperative launch ("global top-k" workloads: the
// whole model is one flat tensor).
//
// Same idea as the general candidate path (sample -> fold + candidates -> select on the
// candidates -> index-ordered emission, exact multi-pass redo as the safety net), specialised:
//   * a CTA owns one column of a row map over the tiles (in the simplest case tiles c, c + G,
//     c + 2G, ... for column c; see RowMap for the unequal shares of large tensors): every CTA
//     sees every region of the tensor, so candidate counts stay balanced even when magnitudes
//     differ between layers;
//   * a CTA appends the candidates of its own tiles to a private, contiguous region of the
//     candidate list (L2-resident) and keeps the per-chunk records in shared memory.  (Holding
//     the candidates themselves in shared memory was measured slower: the large carve-out
//     leaves too little L1 for the streaming loads of the fold pass.);
//   * the sample brackets the threshold from both sides: tau_lo (every element at or above it
//     becomes a candidate) and tau_hi (elements at or above it are almost surely sent).  The
//     fold pass histograms the candidates over [tau_lo, tau_hi) in 2047 equal steps, so after
//     ONE grid barrier every CTA knows the step ("band bin") the k-th largest key lies in;
//   * the few candidates inside that bin go to a short list which every CTA ranks on its own
//     (no further barrier): that gives the exact threshold key and the tie cut;
//   * the fold pass writes +0 into the residual only for candidates at or above tau_z, the
//     sample's estimate of the threshold itself, and a = g + r for the others; the emission
//     then has to touch the residual only where that guess was wrong (a sent candidate below
//     tau_z, an unsent one above it) -- few scattered stores instead of one per unsent candidate;
//   * counting and emission are passes over the CTA's own candidate list, one candidate per
//     thread: the chunk a candidate came from follows from its index, and its output slot is
//     the first slot of that chunk + the sent candidates before it in the chunk (a bit mask in
//     shared memory);
//   * every histogram is flushed to global memory and, after the grid barrier, EVERY CTA scans
//     it and derives the same result -- no completion counters, no designated CTA;
//   * output slots come from per-row totals: row i holds the i-th tile of every column.
// Nothing here is probabilistic in its result: the counts decide, and whenever the bracket
// misses (or a list overflows) the exact multi-pass kernels redo the tensor.
#pragma once
#include "gc_fast.cuh"

namespace gc {

// Fine sample bins per coarse bin, log2.  7 gives tau 18 significant bits; measured on the
// 110M-element workload the step got faster from 5 to 7 bits (fewer collisions between the
// sample's global atomics) and no faster beyond.
constexpr int kFineBits = 7;
constexpr int kFineShift = 31 - 11 - kFineBits;        // key >> kFineShift = fine bin
constexpr uint32_t kFineBins = 1u << (11 + kFineBits);
// Neighbouring fine bins are the hot ones (most samples fall into a few binades), so their
// counters are spread over distinct cache lines: slot = bin * odd constant mod kFineBins.
__device__ __forceinline__ uint32_t fine_slot(uint32_t bin) { return (bin * 40503u) & (kFineBins - 1u); }
constexpr uint32_t kMidRegs = 4;                       // short-list entries a thread keeps in registers
constexpr uint32_t kMidFast = kMidRegs * kBlock;       // short lists up to this size are read once

// Rows of tiles.  A column is one CTA's share of the tensor: row i of column c is one tile, and
// the tiles are numbered row by row.  The three CTAs that share an SM do not advance at the same
// speed (the oldest one gets the most issue slots: with equal shares the first finished its fold
// pass at 182 us, the third at 209 us on the 110M-element workload), so the columns come in
// three classes of gA each with n0 >= n1 >= n2 rows, and every CTA takes a column of the class
// that matches its age on its SM.  Row i is G wide below n2, 2 gA wide below n1, gA wide below
// n0.  Plans that do not fill the GPU three CTAs deep use one class (gA = G, n0 = n1 = n2).
struct RowMap {
    uint32_t G, gA, n0, n1, n2;
    uint32_t s1, s2;                 // first tile of row n2 and of row n1
    uint32_t mG, m2A, mA;            // floor(2^32 / d) + 1 for d = G, 2 gA, gA: t / d = mulhi(t, m) for t < 2^20
    __device__ __forceinline__ uint32_t rows_of(uint32_t c) const { return c < gA ? n0 : c < 2u * gA ? n1 : n2; }
    __device__ __forceinline__ uint32_t tile_of(uint32_t i, uint32_t c) const {
        return i < n2 ? i * G + c : i < n1 ? s1 + (i - n2) * 2u * gA + c : s2 + (i - n1) * gA + c;
    }
    __device__ __forceinline__ void locate(uint32_t t, uint32_t& row, uint32_t& col) const {
        if (t < s1) { row = __umulhi(t, mG); col = t - row * G; }
        else if (t < s2) { const uint32_t q = __umulhi(t - s1, m2A); row = n2 + q; col = t - s1 - q * 2u * gA; }
        else { const uint32_t q = __umulhi(t - s2, mA); row = n1 + q; col = t - s2 - q * gA; }
    }
    __device__ __forceinline__ uint32_t row_of(uint32_t t) const {
        return t < s1 ? __umulhi(t, mG) : t < s2 ? n2 + __umulhi(t - s1, m2A) : n1 + __umulhi(t - s2, mA);
    }
};

// This CTA's arrival number on its SM (0 = it got there first) and the SM's number; the counters
// are zeroed before the launch.
__device__ __forceinline__ uint32_t note_age(uint32_t* per_sm, uint32_t& smid) {
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    return atomicAdd(per_sm + (smid & 1023u), 1u);
}
// Column of this CTA once every CTA has called note_age (after a grid barrier): by age, oldest
// first, column = age x gA + SM number.  That is a one-to-one assignment only if SMs 0..gA-1
// hold three CTAs each; every CTA checks the same counters and otherwise keeps column b.
// Called by the whole CTA (contains a block-wide vote).
__device__ __forceinline__ uint32_t aged_column(const RowMap& rm, const uint32_t* per_sm, uint32_t age, uint32_t smid,
                                                uint32_t G, uint32_t b, int tid) {
    const bool fits = (uint32_t)tid >= rm.gA || ld_cg(per_sm + tid) == 3u;
    const bool none_beyond = (uint32_t)tid < rm.gA || tid >= 1024 || ld_cg(per_sm + tid) == 0u;
    const bool aged = __syncthreads_and(fits && none_beyond) && rm.gA * 3u == G && rm.gA <= (uint32_t)kBlock;
    return aged ? min(age, 2u) * rm.gA + smid : b;
}

struct SingleArgs {
    TensorDesc d;                    // the tensor (by value)
    const TensorDesc* desc;          // device table (for the redo phases)
    uint32_t ntiles, maxt, pool_cap; // tiles, max tiles per CTA, pool slots per CTA
    RowMap rows;                     // which tile is row i of column c
    uint32_t srank_hi;               // sample rank of the upper bracket (at least 1)
    uint32_t srank_mid;              // sample rank that estimates the threshold itself
    uint32_t mid_cap;                // capacity of the short list
    const void* g;                   // fp32 or bf16, see the kernel's template argument
    float* r;
    uint32_t* out_idx;
    float* out_val;
    uint32_t* out_count;
    uint2* cand;                     // [gridDim.x * pool_cap] candidate list, one region per CTA
    uint2* mid;                      // [mid_cap] candidates inside the band bin of the threshold
    uint32_t* hist5;                 // [0] coarse sample histogram, [2] band histogram,
                                     // [3][0] short-list length (all zeroed)
    uint32_t* age;                   // [1024] CTAs that have arrived on every SM (zeroed)
    uint32_t* fine;                  // [kFineBins] fine sample histogram (zeroed)
    uint32_t* tile_cnt;              // [ntiles] candidates above the band bin, per tile
    uint32_t* seg_tot;               // [maxt][ceil(G/32)] the same summed over each run of 32 CTAs of a row (zeroed)
    WsView ws, gws;
    CleanArgs cl;                    // the control block is left clean for the next launch
};


__device__ __forceinline__ void flush_hist(BlockSmem& sm, uint32_t* hist, int nb) {
    __syncthreads();
    for (int b = threadIdx.x; b < nb; b += kBlock) {
        uint32_t c = sm.hist[b];
        if (c) { atomicAdd(hist + b, c); sm.hist[b] = 0u; }
    }
}

// NR ranks (1 = largest; 0 = not wanted) in one histogram of NB bins that is read once from
// global memory.  For each: the bin that holds the rank, the count above the bin and the count
// inside it; ok = the histogram holds at least that many entries.
struct Picked { uint32_t bin, above, count; bool ok; };
template <int NB, int NR>
__device__ void block_select_multi(BlockSmem& sm, const uint32_t* hist, const uint32_t (&k)[NR], Picked (&p)[NR]) {
    static_assert(NR <= kWarps, "results live in per-warp slots");
    constexpr int BPT = (NB + kBlock - 1) / kBlock;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t c[BPT], sum = 0;
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        const int b = NB - 1 - (tid * BPT + i);
        c[i] = b >= 0 ? ld_cg(hist + b) : 0u;
        sum += c[i];
    }
    const uint32_t inc = warp_incl_scan(sum, lane);
    __syncthreads();
    if (lane == 31) sm.scratch[warp] = inc;
    if (tid < NR) sm.gt_tot[tid] = 0xFFFFFFFFu;
    __syncthreads();
    if (warp == 0) {
        const uint32_t v = lane < kWarps ? sm.scratch[lane] : 0u;
        const uint32_t wi = warp_incl_scan(v, lane);
        if (lane < kWarps) sm.scratch[lane] = wi - v;
        if (lane == kWarps - 1) sm.scratch[kWarps] = wi;
    }
    __syncthreads();
    uint32_t above = sm.scratch[warp] + inc - sum;
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        const int b = NB - 1 - (tid * BPT + i);
        if (b >= 0) {
#pragma unroll
            for (int r = 0; r < NR; ++r)
                if (above < k[r] && k[r] <= above + c[i]) { sm.gt_tot[r] = (uint32_t)b; sm.eq_tot[r] = above; sm.gt_ex[r] = c[i]; }
        }
        above += c[i];
    }
    __syncthreads();
    const uint32_t total = sm.scratch[kWarps];
#pragma unroll
    for (int r = 0; r < NR; ++r) {
        p[r].bin = sm.gt_tot[r]; p[r].above = sm.eq_tot[r]; p[r].count = sm.gt_ex[r];
        p[r].ok = k[r] != 0u && total >= k[r] && p[r].bin != 0xFFFFFFFFu;
    }
    __syncthreads();
}

// The same for ONE rank by ONE warp (all 32 lanes call): the 2048 bins are read once with sixteen
// coalesced 16-byte loads per lane, so the eight warps of a CTA can each settle a different
// histogram at the same time, without a block-wide barrier.  Lane l holds, in round i, the four
// bins 4 (32 i + l) .. + 3; a "row" is the 128 bins of one round.
__device__ __forceinline__ Picked warp_select_2048(const uint32_t* hist, uint32_t k, int lane) {
    uint32_t rows[16], total = 0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {                        // eight loads in flight at a time (registers)
        uint4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = ld_cg(reinterpret_cast<const uint4*>(hist) + 32 * (8 * h + i) + lane);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            rows[8 * h + i] = __reduce_add_sync(0xFFFFFFFFu, v[i].x + v[i].y + v[i].z + v[i].w);
            total += rows[8 * h + i];
        }
    }
    Picked p; p.bin = 0xFFFFFFFFu; p.above = 0u; p.count = 0u; p.ok = false;
    if (k == 0u || total < k) return p;
    // the row that holds the rank, from the top, and the count above that row
    uint32_t above = 0; int R = -1;
#pragma unroll
    for (int i = 15; i >= 0; --i)
        if (R < 0) { if (above + rows[i] >= k) R = i; else above += rows[i]; }
    const uint4 vr = ld_cg(reinterpret_cast<const uint4*>(hist) + 32 * R + lane);      // (that row once more)
    // inside the row, lanes from the top: position q stands for lane 31 - q
    const uint32_t mine = vr.x + vr.y + vr.z + vr.w;
    const uint32_t t = __shfl_sync(0xFFFFFFFFu, mine, 31 - lane);
    const uint32_t inc = warp_incl_scan(t, lane);
    const unsigned hit = __ballot_sync(0xFFFFFFFFu, above + inc >= k);
    const int q = __ffs(hit) - 1;                                          // (hit != 0: the row holds the rank)
    const uint32_t above_l = above + __shfl_sync(0xFFFFFFFFu, inc - t, q);
    const int L = 31 - q;
    const uint32_t c3 = __shfl_sync(0xFFFFFFFFu, vr.w, L), c2 = __shfl_sync(0xFFFFFFFFu, vr.z, L);
    const uint32_t c1 = __shfl_sync(0xFFFFFFFFu, vr.y, L), c0 = __shfl_sync(0xFFFFFFFFu, vr.x, L);
    const uint32_t base = 4u * (32u * (uint32_t)R + (uint32_t)L);
    uint32_t ab = above_l;
    if (ab + c3 >= k) { p.bin = base + 3u; p.count = c3; }
    else { ab += c3;
        if (ab + c2 >= k) { p.bin = base + 2u; p.count = c2; }
        else { ab += c2;
            if (ab + c1 >= k) { p.bin = base + 1u; p.count = c1; }
            else { ab += c1; p.bin = base; p.count = c0; } } }
    p.above = ab; p.ok = true;
    return p;
}

// Rank `rank` (1 = largest) among the values f(entry) of the short-list entries that f accepts,
// by radix select over `nbits` bits, 11 at a time from the top, with the histogram in shared
// memory.  Every CTA runs this on the same list and gets the same answer.  Entries come from
// registers (e[], the first kMidFast) and from global memory beyond them.  Returns false if
// fewer than `rank` entries are accepted; `above` = accepted entries with a larger value,
// `at` = accepted entries with exactly the selected value.  sm.hist must be zero on entry and
// is zero again on return.
template <typename F>
__device__ bool short_list_select(BlockSmem& sm, const uint2 (&e)[kMidRegs], const uint2* mid, uint32_t m,
                                  int nbits, uint32_t rank, F f, uint32_t& value, uint32_t& above,
                                  uint32_t& at) {
    const int tid = threadIdx.x;
    uint32_t prefix = 0, krem = rank;
    above = 0; at = 0;
    bool ok = true;
    for (int hi = nbits; hi > 0 && ok; hi -= 11) {
        const int lo = hi > 11 ? hi - 11 : 0, w = hi - lo;          // this level: bits [lo, hi)
        auto count = [&](const uint2& pr) {
            uint32_t v;
            if (!f(pr, v)) return;
            if (hi < 32 && (v >> hi) != prefix) return;
            atomicAdd(&sm.hist[(v >> lo) & ((1u << w) - 1u)], 1u);
        };
#pragma unroll
        for (uint32_t u = 0; u < kMidRegs; ++u)
            if (u * kBlock + tid < m) count(e[u]);
        for (uint32_t i = kMidFast + tid; i < m; i += kBlock) count(ld_cg(mid + i));
        __syncthreads();
        uint32_t bin, ab;
        ok = block_select<2048, true>(sm, sm.hist, krem, bin, ab);
        at = ok ? sm.hist[bin] : 0u;
        __syncthreads();
        for (int i = tid; i < 2048; i += kBlock) sm.hist[i] = 0u;
        __syncthreads();
        if (ok) { prefix = (prefix << w) | bin; krem -= ab; above += ab; }
    }
    value = prefix;
    return ok;
}

// Three CTAs per SM (80 registers, no spills): measured 15 us faster on the 110M-element workload
// than four CTAs at 64 registers with spills, and than two.
template <typename GL>
static __global__ void __launch_bounds__(kBlock, 3)
k_topk_single(const __grid_constant__ SingleArgs a) {
    __shared__ BlockSmem sm;
    __shared__ uint32_t s_used;
    extern __shared__ __align__(16) unsigned char s_dyn[];
    // dynamic shared memory: chunk records, per-chunk counts, output slot of every own tile
    uint32_t* const rec = reinterpret_cast<uint32_t*>(s_dyn);                  // [maxt*kWarps] off<<10 | cnt
    uint32_t* const rec2 = rec + (size_t)a.maxt * kWarps;                      // [maxt*kWarps] above the band bin
    uint32_t* const tile_base = rec2 + (size_t)a.maxt * kWarps;                // [maxt]
    uint32_t* const row_sum = tile_base + a.maxt;                              // [maxt]
    uint32_t* const row_mid = row_sum + a.maxt;                                // [maxt]
    uint32_t* const sent_bits = row_mid + a.maxt;                              // [ceil(pool_cap / 32)]
    // This CTA's region.  Only this CTA (hence only this SM) ever writes or reads it, and it is
    // never read before it is written, so the later phases may read it through L1.
    uint2* const pool = a.cand + (size_t)blockIdx.x * a.pool_cap;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t G = gridDim.x, b = blockIdx.x;
    const TensorDesc& d = a.d;
    WsHeader* hdr = a.ws.hdr;
    uint32_t passed = 0, n_stamp = 0;
    const RowMap& rm = a.rows;
    __shared__ uint32_t s_age[2];
    // This CTA's age among the CTAs of its SM = its arrival number at the SM's counter, taken
    // first thing: the number has to reflect the order in which the CTAs really started (a load
    // in front of it was measured to cost the fold pass 10 us: the shares no longer matched).
    uint32_t my_age = 0, my_sm = 0;
    if (tid == 0) my_age = note_age(a.age, my_sm);
    if (!clean_begin(a.cl, hdr, G, b, tid)) return;
    for (int i = tid; i < 2048; i += kBlock) sm.hist[i] = 0u;
    for (uint32_t i = tid; i < a.maxt * kWarps; i += kBlock) rec2[i] = 0u;
    for (uint32_t i = tid; i < a.maxt; i += kBlock) row_mid[i] = 0u;
    const uint32_t nseg = (G + 31u) / 32u;
    if (tid == 0) s_used = 0u;
    phase_stamp(hdr, n_stamp);

    // ---------------------------------------------------------------- sample
    // One 4-element group out of d.sstride.  Two histograms of the sampled keys are built in one
    // pass: a coarse one (top 11 bits, via shared memory) and a fine one (top 16 bits, straight
    // into global memory; few samples share a fine bin).  tau = the srank-th largest sampled
    // key cut to 16 bits; tau_hi = upper edge of the 16-bit cell of the srank_hi-th largest.
    uint32_t tau = 0, tau_hi = 0x80000000u, tau_z = 0;
    uint32_t col = b, n_own = 0, myseg = 0;      // set after the first barrier
    {
        const uint32_t ngroups = (d.n + 3u) >> 2;
        const uint32_t nsg = (ngroups + d.sstride - 1) / d.sstride;
        constexpr int kMaxOwn = 2;                       // sample groups a thread may own
        uint32_t skey[kMaxOwn][4], sok = 0;
#pragma unroll
        for (int q = 0; q < kMaxOwn; ++q) {
            const uint64_t sg = (uint64_t)q * G * kBlock + (uint64_t)b * kBlock + tid;
            const uint64_t gi = sample_group(sg, d.sstride);
            const bool in = sg < nsg && gi < ngroups;
            const uint32_t i0 = in ? (uint32_t)gi * 4u : 0u;
            float gv[4], rv[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool v = in && i0 + e < d.n;
                const uint32_t f = d.off + (v ? i0 + e : 0u);
                gv[e] = v ? GL::ld1(a.g, f) : 0.f;
                rv[e] = v ? ld_cg(a.r + f) : 0.f;
                sok |= (uint32_t)v << (4 * q + e);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) skey[q][e] = key_of(__fadd_rn(gv[e], rv[e]));
        }
        if (tid == 0) { s_age[0] = my_age; s_age[1] = my_sm; }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kMaxOwn; ++q)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool okq = (sok >> (4 * q + e)) & 1u;
                hist_add_warp(sm.hist, okq ? skey[q][e] >> level_shift(0) : 0xFFFFFFFFu, lane);
                if (okq) atomicAdd(a.fine + fine_slot(skey[q][e] >> kFineShift), 1u);
            }
        // the first own tile is asked into L2 while the sample is being settled
        if (b < a.ntiles) {
            const uint32_t pb = (d.off & ~3u) + b * (uint32_t)kTile + warp * kWarpChunk + lane * 4;
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                if (pb + j * 128 + 4 <= d.off + d.n) {
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(GL::at(a.g, pb + j * 128)));
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(a.r + pb + j * 128));
                }
            }
        }
        flush_hist(sm, a.hist5 + 0 * kHistBins, 1 << level_bits(0));
        if (!grid_barrier(hdr, passed, &sm.ok)) return;
        phase_stamp(hdr, n_stamp);
        clean_in_use(hdr, b, tid);
        {
            col = aged_column(rm, a.age, s_age[0], s_age[1], G, b, tid);
            n_own = rm.rows_of(col);
            while (n_own > 0u && rm.tile_of(n_own - 1u, col) >= a.ntiles) --n_own;
            myseg = col / 32u;
        }
        // both brackets from one read of the coarse histogram, then the kFineBits finer bits of
        // each from the 2^kFineBits fine bins under its coarse bin (one warp per bracket)
        const uint32_t want[3] = {d.srank, a.srank_hi, a.srank_mid};
        Picked pk[3];
        block_select_multi<(1 << level_bits(0)), 3>(sm, a.hist5 + 0 * kHistBins, want, pk);
        if (warp < 3) {
            const Picked& p = pk[warp];
            uint32_t res = 0xFFFFFFFFu;
            if (p.ok) {
                // lane l holds the PER fine bins [top - (l+1) PER, top - l PER) of the coarse bin, highest first
                constexpr uint32_t PER = 1u << (kFineBits - 5);
                const uint32_t first = (p.bin << kFineBits) + (1u << kFineBits) - 1u - (uint32_t)lane * PER;
                uint32_t v[PER], sum = 0;
#pragma unroll
                for (uint32_t j = 0; j < PER; ++j) { v[j] = ld_cg(a.fine + fine_slot(first - j)); sum += v[j]; }
                const uint32_t inc = warp_incl_scan(sum, lane);
                const uint32_t krem = want[warp] - p.above;
                uint32_t mine = 0xFFFFFFFFu, run = inc - sum;
#pragma unroll
                for (uint32_t j = 0; j < PER; ++j) {
                    if (run < krem && krem <= run + v[j]) mine = first - j;
                    run += v[j];
                }
                const unsigned hit = __ballot_sync(0xFFFFFFFFu, mine != 0xFFFFFFFFu);
                if (hit != 0u) res = __shfl_sync(0xFFFFFFFFu, mine, __ffs(hit) - 1);
            }
            if (lane == 0) sm.gt_tot[warp] = res;
        }
        __syncthreads();
        if (sm.gt_tot[0] != 0xFFFFFFFFu) tau = sm.gt_tot[0] << kFineShift;
        if (sm.gt_tot[1] != 0xFFFFFFFFu) tau_hi = (sm.gt_tot[1] + 1u) << kFineShift;
        if (sm.gt_tot[2] != 0xFFFFFFFFu) tau_z = sm.gt_tot[2] << kFineShift;
        __syncthreads();
        // tau == 0 (sample too small for the rank): every element becomes a candidate, the pool
        // overflows and the exact redo takes over
    }
    if (tau_z < tau) tau_z = tau;
    // Band histogram: bin(key) = min((key - tau) >> shift, 2047), monotonic in the key; bins
    // 0..2046 cover [tau, tau_hi) and bin 2047 takes everything above.
    if (tau_hi <= tau) tau_hi = 0x80000000u;
    int shift = 0;
    while (((tau_hi - tau) >> shift) > 2046u) ++shift;

    // ---------------------------------------------------------------- fold + candidates
    const uint32_t my_off = warp * kWarpChunk + lane * 4;
    bool block_overflow = false;
    for (uint32_t i = 0; i < n_own; ++i) {
        const uint32_t tile = rm.tile_of(i, col);
        const TileGeom tg = tile_geom(d, tile);
        const bool interior = tg.lo == tg.base && tg.hi == tg.base + (uint32_t)kTile;
        float av[kVpt][4];
        uint32_t valid = 0xFFFFu;
        if (interior) {
            float4 gv[kVpt], rv[kVpt];
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                gv[j] = GL::ld4(a.g, tg.base + my_off + j * 128);
                rv[j] = ld_cg(reinterpret_cast<const float4*>(a.r + tg.base + my_off + j * 128));
            }
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                av[j][0] = __fadd_rn(gv[j].x, rv[j].x); av[j][1] = __fadd_rn(gv[j].y, rv[j].y);
                av[j][2] = __fadd_rn(gv[j].z, rv[j].z); av[j][3] = __fadd_rn(gv[j].w, rv[j].w);
            }
        } else {
            valid = 0u;
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t f = tg.base + my_off + j * 128 + e;
                    float v = 0.0f;
                    if (f >= tg.lo && f < tg.hi) {
                        v = __fadd_rn(GL::ld1(a.g, f), ld_cg(a.r + f));
                        valid |= 1u << (4 * j + e);
                    }
                    av[j][e] = v;
                }
            }
        }
        uint32_t cnt[kVpt], cm = 0, hm = 0;      // candidates; candidates that are zeroed right away
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
            cnt[j] = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t key = key_of(av[j][e]);
                bool c = key >= tau;
                if (!interior) c = c && ((valid >> (4 * j + e)) & 1u);
                cnt[j] += c;
                cm |= (uint32_t)c << (4 * j + e);
                if (!interior) hm |= (uint32_t)(key >= tau_z) << (4 * j + e);      // tau_z >= tau > 0: implies c
            }
        }
        uint32_t rk[kVpt], wtot;
        warp_rank(cnt, lane, rk, wtot);
        uint32_t off = 0;
        if (lane == 0 && wtot) off = atomicAdd(&s_used, wtot);
        off = __shfl_sync(0xFFFFFFFFu, off, 0);
        const bool fits = off + wtot <= a.pool_cap;
        if (!fits) block_overflow = true;
        if (lane == 0) rec[i * kWarps + warp] = fits ? ((off << 10) | wtot) : 0u;
        const uint32_t em = fits ? cm : 0u;      // goes to the candidate list
        const uint32_t zm = fits ? (hm & cm) : 0u;      // ... and leaves +0 in the residual (probably sent)
        if (interior) {
            // +0 where the key reaches tau_z (implies a candidate: tau_z >= tau), a elsewhere; a chunk that
            // did not fit keeps all its values (no key reaches 2^31)
            const uint32_t tz = fits ? tau_z : 0x80000000u;
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                float4 o;
                o.x = key_of(av[j][0]) >= tz ? 0.0f : av[j][0];
                o.y = key_of(av[j][1]) >= tz ? 0.0f : av[j][1];
                o.z = key_of(av[j][2]) >= tz ? 0.0f : av[j][2];
                o.w = key_of(av[j][3]) >= tz ? 0.0f : av[j][3];
                __stcs(reinterpret_cast<float4*>(a.r + tg.base + my_off + j * 128), o);    // streaming: evict first
            }
        } else {
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if ((valid >> (4 * j + e)) & 1u)
                        a.r[tg.base + my_off + j * 128 + e] = ((zm >> (4 * j + e)) & 1u) ? 0.0f : av[j][e];
                }
            }
        }
        // candidates are ranked into the warp's shared staging row, then written out as one
        // contiguous run of 8-byte pairs
        const bool staged = wtot <= (uint32_t)kEmitStage;
        if (fits && wtot != 0u) {
            // one round per candidate of the lane that has the most (one or two at densities around
            // 1 %), instead of sixteen predicated blocks that every warp walks through
            for (uint32_t m = em; m != 0u; m &= m - 1u) {
                const uint32_t bq = (uint32_t)__ffs((int)m) - 1u, j = bq >> 2;      // element 4 j + e of this thread
                // its value by a select tree (no dynamic register indexing)
                float s8[8], s4[4];
#pragma unroll
                for (int q = 0; q < 8; ++q) s8[q] = (bq & 8u) ? av[2 + q / 4][q % 4] : av[q / 4][q % 4];
#pragma unroll
                for (int q = 0; q < 4; ++q) s4[q] = (bq & 4u) ? s8[4 + q] : s8[q];
                const float s20 = (bq & 2u) ? s4[2] : s4[0], s21 = (bq & 2u) ? s4[3] : s4[1];
                const float v = (bq & 1u) ? s21 : s20;
                const uint32_t rkj = (bq & 8u) ? ((bq & 4u) ? rk[3] : rk[2]) : ((bq & 4u) ? rk[1] : rk[0]);
                const uint32_t pos = rkj + (uint32_t)__popc(em & ((1u << bq) - 1u) & (0xFu << (4u * j)));
                const uint2 pr = make_uint2(tg.base + my_off + j * 128u + (bq & 3u), __float_as_uint(v));
                if (staged) sm.emit[warp][pos] = pr; else pool[off + pos] = pr;
                atomicAdd(&sm.hist[min((key_of(v) - tau) >> shift, 2047u)], 1u);
            }

            if (staged) {
                __syncwarp();
                for (uint32_t q = lane; q < wtot; q += 32) pool[off + q] = sm.emit[warp][q];
                __syncwarp();
            }
        }
    }
    if (__syncthreads_or(block_overflow ? 1 : 0)) {
        if (tid == 0) atomicExch(&hdr->overflow, 1u);
    }
    if (tid == 0) atomicAdd(&hdr->cand_total, min(s_used, a.pool_cap));
    const uint32_t used = s_used;      // read linearly only when no chunk anywhere overflowed
    flush_hist(sm, a.hist5 + 2 * kHistBins, 2048);
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
    // the three early sections have had their last reader (the bracket, right after the first
    // barrier): they are zeroed for the next launch
    clean_early(a.cl, G, b, tid);

    // ---------------------------------------------------------------- band bin of the threshold
    // `good` is the same in every CTA: it only depends on global data read after a barrier
    // the first candidates of the count pass are fetched while the histogram is being read
    constexpr uint32_t kPre = 8;
    uint2 pre[kPre];
#pragma unroll
    for (uint32_t u = 0; u < kPre; ++u) pre[u] = u * kBlock + tid < used ? pool[u * kBlock + tid] : make_uint2(0u, 0u);
    const uint32_t overflowed = ld_cg(&hdr->overflow);
    const uint32_t want_k[1] = {d.k};
    Picked pa[1];
    block_select_multi<2048, 1>(sm, a.hist5 + 2 * kHistBins, want_k, pa);
    const uint32_t A = pa[0].bin, aboveA = pa[0].above, m = pa[0].count;      // m = candidates inside the band bin
    bool good = overflowed == 0u && pa[0].ok && m <= a.mid_cap;

    if (good) {
        // ------------------------------------------------------------ counts above the band bin
        // One linear pass over the CTA's candidates: those above the bin are counted per chunk
        // (the chunk follows from the index), those inside it go to the short list.
        const uint32_t base0 = d.off & ~3u;
        auto classify = [&](const uint2& pr) {
            const uint32_t bin = min(((pr.y & kKeyMask) - tau) >> shift, 2047u);
            if (bin > A) {
                const uint32_t rel = pr.x - base0;
                atomicAdd(&rec2[rm.row_of(rel >> 12) * kWarps + ((rel >> 9) & (kWarps - 1u))], 1u);
            } else if (bin == A) {
                const uint32_t slot = atomicAdd(a.hist5 + 3 * kHistBins, 1u);
                if (slot < a.mid_cap) a.mid[slot] = pr;
            }
        };
#pragma unroll
        for (uint32_t u = 0; u < kPre; ++u)
            if (u * kBlock + tid < used) classify(pre[u]);
        for (uint32_t i0 = kPre * kBlock + tid; i0 < used; i0 += 4 * kBlock) {      // four loads in flight per thread
            uint2 pr[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t i = i0 + u * kBlock;
                pr[u] = i < used ? pool[i] : make_uint2(0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (i0 + u * kBlock < used) classify(pr[u]);
        }
        __syncthreads();
        for (uint32_t i = tid; i < n_own; i += kBlock) {
            uint32_t tot = 0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) tot += rec2[i * kWarps + w];
            a.tile_cnt[rm.tile_of(i, col)] = tot;
            atomicAdd(a.seg_tot + (size_t)i * nseg + myseg, tot);
        }
        if (!grid_barrier(hdr, passed, &sm.ok)) return;
        phase_stamp(hdr, n_stamp);

        // ------------------------------------------------------------ exact threshold from the short list
        // Every CTA ranks the same m entries: Tkey = the (k - aboveA)-th largest key among them.
        // If more entries equal Tkey than are still wanted, the lowest indices win: idx_cut is
        // the largest index that is still sent.
        uint2 e[kMidRegs];
#pragma unroll
        for (uint32_t u = 0; u < kMidRegs; ++u)
            e[u] = u * kBlock + tid < m ? ld_cg(a.mid + u * kBlock + tid) : make_uint2(0u, 0u);
        // while those loads fly: per row, the candidates above the bin in the whole row and in
        // the tiles of lower CTAs (whole 32-CTA segments below this CTA's + the lower CTAs of
        // its own segment): two loads per lane and row, two rows per step
        for (uint32_t i0 = warp * 2u; i0 < n_own; i0 += kWarps * 2u) {
            uint32_t sv[2], tv[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const uint32_t i = i0 + u, q = myseg * 32u + (uint32_t)lane;
                sv[u] = (i < n_own && (uint32_t)lane < nseg) ? ld_cg(a.seg_tot + (size_t)i * nseg + lane) : 0u;
                tv[u] = (i < n_own && q < col) ? ld_cg(a.tile_cnt + rm.tile_of(i, q)) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const uint32_t row = __reduce_add_sync(0xFFFFFFFFu, sv[u]);
                const uint32_t low = __reduce_add_sync(0xFFFFFFFFu, tv[u] + ((uint32_t)lane < myseg ? sv[u] : 0u));
                if (lane == 0 && i0 + u < n_own) { row_sum[i0 + u] = row; tile_base[i0 + u] = low; }
            }
        }
        const uint32_t binlo = tau + (A << shift);
        uint32_t v_sel, mid_gt, n_eq, idx_cut = 0xFFFFFFFFu;
        good = short_list_select(sm, e, a.mid, m, A == 2047u ? 31 : max(shift, 1), d.k - aboveA,
                                 [&](const uint2& pr, uint32_t& v) { v = (pr.y & kKeyMask) - binlo; return true; },
                                 v_sel, mid_gt, n_eq);
        const uint32_t Tkey = binlo + v_sel;
        const uint32_t m_eq = d.k - aboveA - mid_gt;      // entries equal to Tkey that are sent
        if (good && n_eq > m_eq && n_eq <= (uint32_t)kBlock) {
            // a few entries tie at the threshold: list their indices, rank them directly
            auto note = [&](const uint2& pr) {
                if ((pr.y & kKeyMask) == Tkey) sm.hist[atomicAdd(&sm.hist[2047], 1u)] = pr.x;
            };
#pragma unroll
            for (uint32_t u = 0; u < kMidRegs; ++u)
                if (u * kBlock + tid < m) note(e[u]);
            for (uint32_t i = kMidFast + tid; i < m; i += kBlock) note(ld_cg(a.mid + i));
            __syncthreads();
            if ((uint32_t)tid < n_eq) {
                const uint32_t mine = sm.hist[tid];
                uint32_t lower = 0;
                for (uint32_t j = 0; j < n_eq; ++j) lower += sm.hist[j] < mine;
                if (lower == m_eq - 1u) sm.scratch[0] = mine;
            }
            __syncthreads();
            idx_cut = sm.scratch[0];
            __syncthreads();
            if ((uint32_t)tid < n_eq) sm.hist[tid] = 0u;
            if (tid == 0) sm.hist[2047] = 0u;
            __syncthreads();
        } else if (good && n_eq > m_eq) {
            uint32_t v_idx, x0, x1;
            good = short_list_select(sm, e, a.mid, m, 32, m_eq,
                                     [&](const uint2& pr, uint32_t& v) { v = ~pr.x; return (pr.y & kKeyMask) == Tkey; },
                                     v_idx, x0, x1);
            idx_cut = ~v_idx;
        }
        // (a failure here would mean the short list changed under us; all CTAs see the same)
        if (good) {
            // -------------------------------------------------------- output slots
            // A sent short-list entry in tile t raises the slot of every own tile after t, i.e.
            // of the rows from t / G on (one later unless t belongs to a lower CTA); in an own
            // tile it also raises the count of its chunk.
            auto sent_key = [&](const uint2& pr) {
                const uint32_t key = pr.y & kKeyMask;
                return key > Tkey || (key == Tkey && pr.x <= idx_cut);
            };
            auto below = [&](const uint2& pr) {
                if (!sent_key(pr)) return;
                const uint32_t rel = pr.x - base0;
                uint32_t row, owner;
                rm.locate(rel >> 12, row, owner);
                const uint32_t first = row + (owner < col ? 0u : 1u);
                if (first < n_own) atomicAdd(&row_mid[first], 1u);
                if (owner == col) atomicAdd(&rec2[row * kWarps + ((rel >> 9) & (kWarps - 1u))], 1u);
            };
#pragma unroll
            for (uint32_t u = 0; u < kMidRegs; ++u)
                if (u * kBlock + tid < m) below(e[u]);
            for (uint32_t i = kMidFast + tid; i < m; i += kBlock) below(ld_cg(a.mid + i));
            __syncthreads();
            if (warp == 0) {
                // tile_base[i] = rows before i + lower CTAs of row i + sent short-list entries before the tile
                uint32_t run = 0;
                for (uint32_t i0 = 0; i0 < n_own; i0 += 32) {
                    const uint32_t i = i0 + lane;
                    const uint32_t v = i < n_own ? row_sum[i] : 0u;
                    const uint32_t w = i < n_own ? row_mid[i] : 0u;
                    const uint32_t inc = warp_incl_scan(v + w, lane);
                    if (i < n_own) tile_base[i] += run + inc - v;
                    run += __shfl_sync(0xFFFFFFFFu, inc, 31);
                }
            }
            __syncthreads();
            // rec2[c] = output slot of the first sent candidate of chunk c
            for (uint32_t i = tid; i < n_own; i += kBlock) {
                uint32_t pos = tile_base[i];
#pragma unroll
                for (int w = 0; w < kWarps; ++w) {
                    const uint32_t c = rec2[i * kWarps + w];
                    rec2[i * kWarps + w] = pos;
                    pos += c;
                }
            }
            phase_stamp(hdr, n_stamp);      // threshold and output slots known
            // sent flags of the CTA's candidates in list order, one bit each
            const uint32_t nwords = (used + 31u) >> 5;
            for (uint32_t i0 = 0; i0 < nwords * 32u; i0 += 4 * kBlock) {
                uint2 pr[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t i = i0 + u * kBlock + tid;
                    pr[u] = i < used ? pool[i] : make_uint2(0u, 0u);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t i = i0 + u * kBlock + tid;
                    if (i0 + u * kBlock + (tid & ~31) >= nwords * 32u) continue;          // whole warp past the end
                    const unsigned sb = __ballot_sync(0xFFFFFFFFu, i < used && sent_key(pr[u]));
                    if (lane == 0) sent_bits[i >> 5] = sb;
                }
            }
            __syncthreads();
            // emission: slot = first slot of the chunk + sent candidates before this one in the chunk
            for (uint32_t i0 = tid; i0 < used; i0 += 4 * kBlock) {
                uint2 pr[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t i = i0 + u * kBlock;
                    pr[u] = i < used ? pool[i] : make_uint2(0u, 0u);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t i = i0 + u * kBlock;
                    if (i >= used) continue;
                    // the fold pass left +0 in the residual iff the key reached tau_z
                    const bool zeroed = (pr[u].y & kKeyMask) >= tau_z;
                    if (!sent_key(pr[u])) {
                        if (zeroed) a.r[pr[u].x] = __uint_as_float(pr[u].y);     // value goes back
                        continue;
                    }
                    if (!zeroed) a.r[pr[u].x] = 0.0f;
                    const uint32_t rel = pr[u].x - base0;
                    const uint32_t c = rm.row_of(rel >> 12) * kWarps + ((rel >> 9) & (kWarps - 1u));
                    const uint32_t s = rec[c] >> 10;                   // first list position of the chunk
                    uint32_t before;
                    if ((s >> 5) == (i >> 5)) {
                        before = __popc((sent_bits[i >> 5] & ((1u << (i & 31u)) - 1u)) >> (s & 31u));
                    } else {
                        before = __popc(sent_bits[s >> 5] >> (s & 31u)) + __popc(sent_bits[i >> 5] & ((1u << (i & 31u)) - 1u));
                        for (uint32_t w = (s >> 5) + 1u; w < (i >> 5); ++w) before += __popc(sent_bits[w]);
                    }
                    const uint32_t slot = rec2[c] + before;
                    if (slot < d.cap) {
                        __stcs(a.out_idx + d.out_off + slot, pr[u].x);
                        __stcs(a.out_val + d.out_off + slot, __uint_as_float(pr[u].y));
                    } else {
                        record_status(hdr, -1 /*GC_E_INVALID*/, pr[u].x);
                    }
                }
            }
            if (a.out_count != nullptr && b == 0 && tid == 0) { a.out_count[0] = d.k; a.out_count[1] = d.k; }
            __syncthreads();
            phase_stamp(hdr, n_stamp);
            exit_stamp(hdr);
            leave_clean(a.cl, hdr, G, tid);
            return;
        }
    }

    // ---------------------------------------------------------------- safety net (rare)
    // The pool overflowed or the candidate set was smaller than k: give every pooled candidate
    // its value back, then run the exact multi-pass kernels on r (= a everywhere again).
    if (b == 0 && tid == 0) { a.ws.sel[0].flags = kSelFailed; atomicAdd(&hdr->n_failed, 1u); }
    for (uint32_t c = tid; c < n_own * kWarps; c += kBlock) {      // only chunks that were stored
        const uint32_t rc = rec[c], off = rc >> 10, cnt = rc & 1023u;
        for (uint32_t j = 0; j < cnt; ++j) {
            const uint2 pr = pool[off + j];
            a.r[pr.x] = __uint_as_float(pr.y);
        }
    }
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
    hist_body<0, SRC_RESID>(sm, a.desc, 1u, a.ntiles, nullptr, a.r, a.gws);
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    hist_body<1, SRC_RESID>(sm, a.desc, 1u, a.ntiles, nullptr, a.r, a.gws);
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    hist_body<2, SRC_RESID>(sm, a.desc, 1u, a.ntiles, nullptr, a.r, a.gws);
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    compact_body(sm, a.desc, 1u, a.ntiles, a.r, a.out_idx, a.out_val, a.out_count, a.gws, 0);
    __syncthreads();
    leave_clean(a.cl, hdr, G, tid);
}

}  // namespace gc
