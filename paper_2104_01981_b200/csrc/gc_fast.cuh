// One-pass candidate path for exact top-k.
//
// A small strided sample of a = g + r gives, per tensor, a key tau_lo that is safely below
// the k-th largest key.  The single full-size pass then folds the residual (12 bytes per
// element) and copies every element with key >= tau_lo into a candidate list (a few per cent
// of the data) while building the first radix histogram of the candidates.  The exact k-th
// key is resolved on the candidate list alone and the final, index-ordered compaction reads
// only candidates.  If the candidate set of a tensor turns out smaller than k, or the list
// overflows, that tensor (or every tensor) is redone by the exact multi-pass kernels, so the
// result never depends on the sample.
//
// Candidate list layout: each warp of the fold pass owns a 512-element chunk of every tile it
// visits and appends that chunk's candidates, in index order, to a slab of kSlab slots it
// reserved with one atomic; chunk_info[tile * kWarps + warp] = (first slot, count).  Chunks
// land in arbitrary order in the list; readers walk them by (tile, warp), which is index order.
//
// All phases exist as __device__ bodies.  k_compress_fused runs them back to back in ONE
// cooperative launch with grid barriers in between; the k_* wrappers run them as separate
// launches (same results, used when a cooperative launch is not wanted).
#pragma once
#include "gc_kernels.cuh"

namespace gc {

struct CandView {
    uint2* pair;             // [cap] (flat index, bits of a = g + r) of each candidate
    uint2* chunk_info;       // [ntiles * kWarps] (first slot, count) per warp chunk
    unsigned long long* group_cnt;   // [ngroups] (above-T << 31 | equal-T) counts per compaction group
    uint32_t cap;
    const TensorSel* ssel;   // [n_tensors] sample selection record (21-bit prefix = tau_lo >> 10)
};

// The candidates of one tile as seen by a warp: lane l < kWarps holds chunk l.
struct TileCands {
    uint32_t base, cnt, incl, total;
};
__device__ __forceinline__ TileCands load_tile_cands(const CandView& cv, uint32_t tile, int lane) {
    TileCands tc;
    uint2 info = make_uint2(0u, 0u);
    if (lane < kWarps) info = ld_cg(&cv.chunk_info[(size_t)tile * kWarps + lane]);
    tc.base = info.x; tc.cnt = info.y;
    tc.incl = warp_incl_scan(tc.cnt, lane);
    tc.total = __shfl_sync(0xFFFFFFFFu, tc.incl, 31);
    return tc;
}
// slot of the j-th candidate of the tile (all lanes call; j >= total gives a harmless slot)
__device__ __forceinline__ uint32_t cand_slot(const TileCands& tc, uint32_t j) {
    uint32_t c = 0;
#pragma unroll
    for (int l = 0; l < kWarps; ++l) c += (j >= __shfl_sync(0xFFFFFFFFu, tc.incl, l)) ? 1u : 0u;
    c = min(c, (uint32_t)kWarps - 1u);
    uint32_t b = __shfl_sync(0xFFFFFFFFu, tc.base, c);
    uint32_t ex = __shfl_sync(0xFFFFFFFFu, tc.incl - tc.cnt, c);
    return b + (j - ex);
}

// ----------------------------------------------------------------------------- small tensors
// Exact top-k of one small tensor (fewer than kSmallMax elements: it fits one tile) by ONE CTA,
// start to finish: the tile is read once and stays in registers through the three histogram
// levels (shared memory, __syncthreads only) and the ordered emission, so hundreds of tiny
// tensors cost one memory round trip each, no global atomics, no completion counters and no
// grid barriers.
template <typename GL = GradF32>
static __device__ __noinline__ void small_tensor_body(BlockSmem& sm, const TensorDesc& d, uint32_t t, uint32_t T,
                                         const void* __restrict__ g, float* __restrict__ r,
                                         uint32_t* __restrict__ out_idx, float* __restrict__ out_val,
                                         uint32_t* __restrict__ out_count) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const TileGeom tg = tile_geom(d, 0u);
    Tile tl;
    load_tile<true, GL>(g, r, tg, warp, lane, tl);           // r = a = g + r; sent entries get +0 below
    uint32_t prefix = 0, krem = d.k;
#pragma unroll 1
    for (int level = 0; level < kLevels; ++level) {
        const int bits = level_bits(level), sh = level_shift(level);
        __syncthreads();
        for (int b = tid; b < (1 << level_bits(0)); b += kBlock) sm.hist[b] = 0u;
        __syncthreads();
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t key = key_of(tl.a[j][e]);
                bool in = (tl.valid >> (4 * j + e)) & 1u;
                if (level > 0) in = in && ((key >> (sh + bits)) == prefix);
                if (level == 0) hist_add_warp(sm.hist, in ? key >> sh : 0xFFFFFFFFu, lane);    // (crowded coarse bins)
                else if (in) atomicAdd(&sm.hist[(key >> sh) & ((1u << bits) - 1u)], 1u);
            }
        }
        __syncthreads();
        uint32_t bin, above;
        if (level == 0) block_select<(1 << level_bits(0)), true>(sm, sm.hist, krem, bin, above);
        else block_select<(1 << level_bits(1)), true>(sm, sm.hist, krem, bin, above);
        prefix = (prefix << bits) | bin;
        krem -= above;
    }
    const uint32_t Tkey = prefix, m_eq = krem;
    // ordered emission
    uint32_t cg[kVpt], ce[kVpt], gtm = 0, eqm = 0;
#pragma unroll
    for (int j = 0; j < kVpt; ++j) {
        cg[j] = 0; ce[j] = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint32_t key = key_of(tl.a[j][e]);
            const bool v = (tl.valid >> (4 * j + e)) & 1u;
            const bool gt = v && key > Tkey, eq = v && key == Tkey;
            cg[j] += gt; ce[j] += eq;
            gtm |= (uint32_t)gt << (4 * j + e);
            eqm |= (uint32_t)eq << (4 * j + e);
        }
    }
    uint32_t rg[kVpt], re[kVpt], wg, we;
    warp_rank(cg, lane, rg, wg);
    warp_rank(ce, lane, re, we);
    __syncthreads();
    if (lane == 0) { sm.gt_tot[warp] = wg; sm.eq_tot[warp] = we; }
    __syncthreads();
    scan_warp_totals(sm.gt_tot, sm.gt_ex, &sm.gt_sum, warp, lane);
    if (warp == 1) {
        uint32_t v = lane < kWarps ? sm.eq_tot[lane] : 0u;
        uint32_t inc = warp_incl_scan(v, lane);
        if (lane < kWarps) sm.eq_ex[lane] = inc - v;
        if (lane == 31) sm.eq_sum = inc;
    }
    __syncthreads();
    if ((gtm | eqm) != 0u) {
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
            uint32_t gpos = sm.gt_ex[warp] + rg[j], epos = sm.eq_ex[warp] + re[j];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool gt = (gtm >> (4 * j + e)) & 1u, eq = (eqm >> (4 * j + e)) & 1u;
                if (gt || (eq && epos < m_eq)) {
                    const uint32_t slot = gpos + min(epos, m_eq);
                    const uint32_t f = vec_index(tg.base, warp, lane, j) + e;
                    if (slot < d.cap) {
                        out_idx[d.out_off + slot] = f;
                        out_val[d.out_off + slot] = tl.a[j][e];
                        r[f] = 0.0f;
                    }
                }
                gpos += gt; epos += eq;
            }
        }
    }
    if (out_count != nullptr && tid == 0) { out_count[t] = d.k; out_count[T + t] = d.k; }
    __syncthreads();
}

// Exact top-k of one TINY tensor (at most kTinyMaxN elements, k at most kTinyMaxK) by ONE WARP:
// no shared memory and no block-wide barrier, so the eight warps of a CTA finish eight such
// tensors at once (layer-wise plans hold dozens of normalisation vectors of 64 to 512 elements
// with k = 1).  The tensor is read once (all loads of a lane in flight together) and stays in
// registers, 16 values per lane.  Pass 0 finds the largest key, ties to the lower index; every
// further pass finds the largest entry that comes strictly after the previous winner in that
// order (key descending, index ascending).  The k winners are then ranked by index for the output.
constexpr uint32_t kTinyMaxN = 512, kTinyMaxK = 16;
__host__ __device__ inline bool is_tiny(uint32_t n, uint32_t k) { return n > 0 && n <= kTinyMaxN && k <= kTinyMaxK; }

__device__ __forceinline__ unsigned long long warp_max64(unsigned long long v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, v, d);
        v = o > v ? o : v;
    }
    return v;
}

template <typename GL = GradF32>
static __device__ __noinline__ void tiny_tensor_warp(const uint32_t off, const uint32_t n, const uint32_t k,
                                                     const uint32_t out_off, uint32_t t, uint32_t T,
                                                     const void* __restrict__ g, float* __restrict__ r,
                                                     uint32_t* __restrict__ out_idx, float* __restrict__ out_val,
                                                     uint32_t* __restrict__ out_count, int lane) {
    constexpr int kU = (int)kTinyMaxN / 32;               // values per lane: element i sits in lane i % 32, slot i / 32
    float gv[kU], rv[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const uint32_t i = (uint32_t)lane + 32u * u;
        gv[u] = i < n ? GL::ld1(g, off + i) : 0.f;
        rv[u] = i < n ? r[off + i] : 0.f;
    }
    // order of two entries as one 64-bit compare: key in the high word, ~index in the low one
    // (a real entry is never 0: ~index > 0)
    unsigned long long best = 0ull;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const uint32_t i = (uint32_t)lane + 32u * u;
        gv[u] = __fadd_rn(gv[u], rv[u]);                  // a = g + r
        const unsigned long long o = ((unsigned long long)key_of(gv[u]) << 32) | (unsigned long long)(~i);
        if (i < n && o > best) best = o;
    }
    unsigned long long win = warp_max64(best), mine = 0ull;    // lane j keeps winner j
    if (lane == 0) mine = win;
    for (uint32_t j = 1; j < k; ++j) {
        best = 0ull;
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const uint32_t i = (uint32_t)lane + 32u * u;
            const unsigned long long o = ((unsigned long long)key_of(gv[u]) << 32) | (unsigned long long)(~i);
            if (i < n && o < win && o > best) best = o;
        }
        win = warp_max64(best);
        if ((uint32_t)lane == j) mine = win;
    }
    // rank of winner `lane` among the winners by index (the low words hold ~index: larger = lower index)
    const uint32_t my_ni = (uint32_t)mine;
    uint32_t rank = 0;
    for (uint32_t j = 0; j < k; ++j) {
        const uint32_t o = __shfl_sync(0xFFFFFFFFu, my_ni, (int)j);
        rank += o > my_ni ? 1u : 0u;
    }
    // the pairs: the lane that holds winner j's value writes it at that winner's rank
    uint32_t sent = 0;                                    // bit u: this lane's slot u is a winner
    for (uint32_t j = 0; j < k; ++j) {
        const uint32_t wi = ~__shfl_sync(0xFFFFFFFFu, my_ni, (int)j);
        const uint32_t rk = __shfl_sync(0xFFFFFFFFu, rank, (int)j);
        if ((wi & 31u) == (uint32_t)lane) {
            float v = 0.f;
#pragma unroll
            for (int u = 0; u < kU; ++u) if ((uint32_t)u == (wi >> 5)) v = gv[u];
            out_idx[out_off + rk] = off + wi;
            out_val[out_off + rk] = v;                    // bit copy of a
            sent |= 1u << (wi >> 5);
        }
    }
    // the residual: a everywhere, +0 at the winners
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const uint32_t i = (uint32_t)lane + 32u * u;
        if (i < n) r[off + i] = ((sent >> u) & 1u) ? 0.0f : gv[u];
    }
    if (out_count != nullptr && lane == 0) { out_count[t] = k; out_count[T + t] = k; }
}

// Exact top-k of one small tensor (it fits one tile) with a FEW entries to keep (k <= kFewK), by
// one CTA: the tile is read once and stays in registers; round q finds the largest entry that
// comes strictly after winner q - 1 in the order (key descending, index ascending) -- a scan of
// the thread's 16 values, a warp-wide and a block-wide maximum, ONE barrier per round instead of
// the twenty-odd of the three histogram levels.  The winners are then ranked by index.
constexpr uint32_t kFewK = 8;
template <typename GL = GradF32>
static __device__ __noinline__ void small_tensor_fewk(BlockSmem& sm, const TensorDesc& d, uint32_t t, uint32_t T,
                                                      const void* __restrict__ g, float* __restrict__ r,
                                                      uint32_t* __restrict__ out_idx, float* __restrict__ out_val,
                                                      uint32_t* __restrict__ out_count) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const TileGeom tg = tile_geom(d, 0u);
    Tile tl;
    load_tile<true, GL>(g, r, tg, warp, lane, tl);           // r = a = g + r; the winners get +0 below
    unsigned long long* const slot = reinterpret_cast<unsigned long long*>(sm.hist);     // [2][kWarps], by round parity
    uint32_t* const widx = sm.hist + 4 * kWarps;                                         // [kFewK] winners' flat indices
    __syncthreads();                                         // (whoever used sm.hist before is done)
    unsigned long long win = ~0ull;
    for (uint32_t q = 0; q < d.k; ++q) {
        unsigned long long best = 0ull;                      // order word: key << 32 | ~flat index (never 0)
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t f = vec_index(tg.base, warp, lane, j) + e;
                const unsigned long long o = ((unsigned long long)key_of(tl.a[j][e]) << 32) | (unsigned long long)(~f);
                if (((tl.valid >> (4 * j + e)) & 1u) && o < win && o > best) best = o;
            }
        }
        best = warp_max64(best);
        if (lane == 0) slot[(q & 1u) * kWarps + warp] = best;
        __syncthreads();
        win = 0ull;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) { const unsigned long long o = slot[(q & 1u) * kWarps + w]; win = o > win ? o : win; }
        if (tid == 0) widx[q] = ~(uint32_t)win;
    }
    __syncthreads();                                         // the winners' list is complete; r = a is visible block-wide
    if ((uint32_t)tid < d.k) {
        const uint32_t f = widx[tid];
        uint32_t rank = 0;
        for (uint32_t q = 0; q < d.k; ++q) rank += widx[q] < f ? 1u : 0u;
        out_idx[d.out_off + rank] = f;
        out_val[d.out_off + rank] = ld_cg(r + f);            // bit copy of a (written by the owning thread of this CTA)
        r[f] = 0.0f;
    }
    if (out_count != nullptr && tid == 0) { out_count[t] = d.k; out_count[T + t] = d.k; }
    __syncthreads();
}

// All small tensors of the plan, dealt out to the CTAs round-robin.
static __device__ void small_tensors_body(BlockSmem& sm, const TensorDesc* __restrict__ desc, uint32_t T,
                                          const uint32_t* __restrict__ small_ids, uint32_t n_small,
                                          const float* __restrict__ g, float* __restrict__ r,
                                          uint32_t* __restrict__ out_idx, float* __restrict__ out_val,
                                          uint32_t* __restrict__ out_count) {
    for (uint32_t q = blockIdx.x; q < n_small; q += gridDim.x) {
        const uint32_t t = small_ids[q];
        const TensorDesc d = desc[t];
        small_tensor_body(sm, d, t, T, g, r, out_idx, out_val, out_count);
    }
}

// ----------------------------------------------------------------------------- fold + candidates
// Reads g and r, computes a = g + r, emits candidates and writes the residual back with the
// candidates ALREADY zeroed (their values live in the candidate list): after the selection
// only the few candidates that were not sent need their value restored, instead of every
// sent entry needing a scattered zero.  A chunk whose candidates did not fit in the list keeps
// its values in r.  CTAs take contiguous runs of tiles (plans with many tensors then change
// tensor -- and flush their histogram -- as rarely as possible).  No block-wide barrier in the
// tile loop: every warp ranks and stores the candidates of its own chunk.
static __device__ void fold_cand_body(BlockSmem& sm, const TensorDesc* __restrict__ desc, uint32_t T,
                                      uint32_t ntiles, const float* __restrict__ g, float* __restrict__ r,
                                      const WsView& ws, const CandView& cv) {
    constexpr int NB = 1 << level_bits(0);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t per = (ntiles + gridDim.x - 1) / gridDim.x;
    const uint32_t first = blockIdx.x * per;
    const uint32_t last = min(ntiles, first + per);
    if (first >= last) return;
    for (int b = tid; b < NB; b += kBlock) sm.hist[b] = 0u;
    __syncthreads();

    uint32_t t = find_tensor(desc, T, first);
    TensorDesc d = desc[t];
    uint32_t tau = d.sstride ? (ld_cg(&cv.ssel[t].prefix) << level_shift(1)) : 0u;
    uint32_t tiles_here = 0;
    uint32_t slab_next = 0, slab_left = 0;       // this warp's current slab (warp-uniform)
    const uint32_t my_off = warp * kWarpChunk + lane * 4;

    for (uint32_t tile = first; tile < last; ++tile) {
        if (tile >= d.tile0 + d.ntiles) {
            if (tiles_here) flush_and_select<0, true>(sm, ws, t, tiles_here, d.ntiles, d.k);
            tiles_here = 0;
            t = find_tensor(desc, T, tile);
            d = desc[t];
            tau = d.sstride ? (ld_cg(&cv.ssel[t].prefix) << level_shift(1)) : 0u;
        }
        if (d.kind == kKindSmall) continue;      // finished by its own CTA
        const TileGeom tg = tile_geom(d, tile - d.tile0);
        const bool interior = tg.lo == tg.base && tg.hi == tg.base + (uint32_t)kTile;
        float a[kVpt][4];
        uint32_t valid = 0xFFFFu;
        if (interior) {
            float4 gv[kVpt], rv[kVpt];
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                gv[j] = __ldg(reinterpret_cast<const float4*>(g + tg.base + my_off + j * 128));
                rv[j] = ld_cg(reinterpret_cast<const float4*>(r + tg.base + my_off + j * 128));
            }
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                a[j][0] = __fadd_rn(gv[j].x, rv[j].x); a[j][1] = __fadd_rn(gv[j].y, rv[j].y);
                a[j][2] = __fadd_rn(gv[j].z, rv[j].z); a[j][3] = __fadd_rn(gv[j].w, rv[j].w);
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
                        v = __fadd_rn(__ldg(g + f), ld_cg(r + f));
                        valid |= 1u << (4 * j + e);
                    }
                    a[j][e] = v;
                }
            }
        }
        uint32_t cnt[kVpt], cm = 0;
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
            cnt[j] = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                bool c = key_of(a[j][e]) >= tau;
                if (!interior) c = c && ((valid >> (4 * j + e)) & 1u);
                cnt[j] += c;
                cm |= (uint32_t)c << (4 * j + e);
            }
        }
        uint32_t rk[kVpt], wtot;
        warp_rank(cnt, lane, rk, wtot);
        // reserve slots for this chunk out of the warp's slab (new slab when it runs short)
        bool fits = true;
        if (wtot > slab_left) {
            uint32_t need = max(wtot, (uint32_t)kSlab);
            uint32_t nb = 0;
            if (lane == 0) nb = atomicAdd(&ws.hdr->cand_total, need);
            nb = __shfl_sync(0xFFFFFFFFu, nb, 0);
            if (nb > cv.cap || need > cv.cap - nb) {
                fits = false;
                if (lane == 0) atomicExch(&ws.hdr->overflow, 1u);
                slab_left = 0;
            } else {
                slab_next = nb; slab_left = need;
            }
        }
        const uint32_t cbase = slab_next;
        if (fits) { slab_next += wtot; slab_left -= wtot; }
        if (lane == 0) cv.chunk_info[(size_t)tile * kWarps + warp] = make_uint2(cbase, fits ? wtot : 0u);
        // residual write-back: a, with +0 where the element went into the candidate list
        const uint32_t zm = fits ? cm : 0u;
        if (interior) {
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                float4 o;
                o.x = ((zm >> (4 * j + 0)) & 1u) ? 0.0f : a[j][0];
                o.y = ((zm >> (4 * j + 1)) & 1u) ? 0.0f : a[j][1];
                o.z = ((zm >> (4 * j + 2)) & 1u) ? 0.0f : a[j][2];
                o.w = ((zm >> (4 * j + 3)) & 1u) ? 0.0f : a[j][3];
                *reinterpret_cast<float4*>(r + tg.base + my_off + j * 128) = o;
            }
        } else {
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if ((valid >> (4 * j + e)) & 1u)
                        r[tg.base + my_off + j * 128 + e] = ((zm >> (4 * j + e)) & 1u) ? 0.0f : a[j][e];
                }
            }
        }
        // emission: candidates are first ranked into the warp's shared staging row, then written
        // out as one contiguous run of 8-byte pairs (a chunk rarely holds more than a dozen)
        const bool staged = wtot <= (uint32_t)kEmitStage;
        if (fits && wtot != 0u) {
            if (cm != 0u) {
#pragma unroll
                for (int j = 0; j < kVpt; ++j) {
                    uint32_t pos = rk[j];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if ((cm >> (4 * j + e)) & 1u) {
                            const uint2 pr = make_uint2(tg.base + my_off + j * 128 + e, __float_as_uint(a[j][e]));
                            if (staged) sm.emit[warp][pos] = pr; else cv.pair[cbase + pos] = pr;
                            atomicAdd(&sm.hist[key_of(a[j][e]) >> level_shift(0)], 1u);
                            ++pos;
                        }
                    }
                }
            }
            if (staged) {
                __syncwarp();
                for (uint32_t i = lane; i < wtot; i += 32) cv.pair[cbase + i] = sm.emit[warp][i];
                __syncwarp();
            }
        }
        ++tiles_here;
    }
    if (tiles_here) flush_and_select<0, true>(sm, ws, t, tiles_here, d.ntiles, d.k);
}

// Puts the value of every listed candidate back into the residual, for the tensors that are
// about to be redone by the exact kernels (those need r = a everywhere).
static __device__ void cand_restore_body(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles,
                                         float* __restrict__ r, const WsView& ws, const CandView& cv) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool all = ld_cg(&ws.hdr->overflow) != 0u;
    if (!all && ld_cg(&ws.hdr->n_failed) == 0u) return;
    for (uint32_t tile = blockIdx.x * kWarps + warp; tile < ntiles; tile += gridDim.x * kWarps) {
        const uint32_t t = find_tensor(desc, T, tile);
        if (desc[t].kind == kKindSmall) continue;
        if (!all && (ld_cg(&ws.sel[t].flags) & kSelFailed) == 0u) continue;
        TileCands tc = load_tile_cands(cv, tile, lane);
        for (uint32_t j0 = 0; j0 < tc.total; j0 += 32) {
            uint32_t j = j0 + lane;
            uint32_t slot = cand_slot(tc, j);
            if (j < tc.total) {
                const uint2 pr = ld_cg(&cv.pair[slot]);
                r[pr.x] = __uint_as_float(pr.y);
            }
        }
    }
}

// ----------------------------------------------------------------------------- candidate refinement
// Radix-select level 1 or 2 over the candidate lists.  CTAs take contiguous runs of tiles and
// walk them kWarps at a time, one warp per tile, always inside one tensor; counts go to the
// shared-memory histogram that is flushed when the tensor changes, and the CTA that completes
// a tensor's last tile runs the select step (same scheme as hist_body).
template <int LEVEL>
__device__ void cand_hist_body(BlockSmem& sm, const TensorDesc* __restrict__ desc, uint32_t T,
                               uint32_t ntiles, const WsView& ws, const CandView& cv) {
    constexpr int NB = 1 << level_bits(LEVEL);
    constexpr int SH = level_shift(LEVEL);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t per = (ntiles + gridDim.x - 1) / gridDim.x;
    const uint32_t first = blockIdx.x * per;
    const uint32_t last = min(ntiles, first + per);
    if (first >= last) return;
    for (int b = tid; b < NB; b += kBlock) sm.hist[b] = 0u;
    __syncthreads();

    uint32_t t = find_tensor(desc, T, first);
    TensorDesc d = desc[t];
    bool active = d.kind != kKindSmall && (ld_cg(&ws.sel[t].flags) & kSelFailed) == 0u;
    uint32_t prefix = ld_cg(&ws.sel[t].prefix);
    uint32_t tiles_here = 0;

    uint32_t batch = first;
    while (batch < last) {
        if (batch >= d.tile0 + d.ntiles) {
            if (active && tiles_here) flush_and_select<LEVEL, false>(sm, ws, t, tiles_here, d.ntiles, 0u);
            tiles_here = 0;
            t = find_tensor(desc, T, batch);
            d = desc[t];
            active = d.kind != kKindSmall && (ld_cg(&ws.sel[t].flags) & kSelFailed) == 0u;
            prefix = ld_cg(&ws.sel[t].prefix);
        }
        const uint32_t bend = min(min(last, d.tile0 + d.ntiles), batch + (uint32_t)kWarps);
        const uint32_t tile = batch + warp;
        if (active && tile < bend) {
            TileCands tc = load_tile_cands(cv, tile, lane);
            for (uint32_t j0 = 0; j0 < tc.total; j0 += 32) {
                uint32_t j = j0 + lane;
                uint32_t slot = cand_slot(tc, j);
                if (j < tc.total) {
                    uint32_t key = ld_cg(&cv.pair[slot]).y & kKeyMask;
                    if ((key >> (SH + level_bits(LEVEL))) == prefix)
                        atomicAdd(&sm.hist[(key >> SH) & (NB - 1)], 1u);
                }
            }
        }
        tiles_here += bend - batch;
        batch = bend;
    }
    if (active && tiles_here) flush_and_select<LEVEL, false>(sm, ws, t, tiles_here, d.ntiles, 0u);
}

// ----------------------------------------------------------------------------- candidate compaction
// Index-ordered emission from the candidate lists in two steps.  A group is kWarps consecutive
// tiles of one tensor, one warp per tile; group i of a CTA is blockIdx.x + i * gridDim.x.
//   count: every group stores its (above-T, equal-T) totals;
//   emit:  a group adds up the totals of the groups before it in its tensor, ranks its own
//          candidates, writes the sent ones to the output (their residual is already +0) and
//          restores the value of the others in the residual.
// An element is sent iff key > T, or key == T and fewer than m_eq equal keys precede it.
__device__ __forceinline__ void group_tile_counts(const CandView& cv, const TileCands& tc, uint32_t Tkey,
                                                  int lane, uint32_t& ngt, uint32_t& neq) {
    ngt = 0; neq = 0;
    for (uint32_t j0 = 0; j0 < tc.total; j0 += 32) {
        uint32_t j = j0 + lane;
        uint32_t slot = cand_slot(tc, j);
        uint32_t key = j < tc.total ? (ld_cg(&cv.pair[slot]).y & kKeyMask) : 0u;
        bool gt = j < tc.total && key > Tkey, eq = j < tc.total && key == Tkey;
        ngt += __popc(__ballot_sync(0xFFFFFFFFu, gt));
        neq += __popc(__ballot_sync(0xFFFFFFFFu, eq));
    }
}

template <bool EMIT>
__device__ void cand_compact_body(BlockSmem& sm, const TensorDesc* __restrict__ desc, uint32_t T,
                                  uint32_t ngroups_total, float* __restrict__ r,
                                  uint32_t* __restrict__ out_idx, float* __restrict__ out_val,
                                  uint32_t* __restrict__ out_count, const WsView& ws, const CandView& cv) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned lt_mask = (1u << lane) - 1u;
    for (uint32_t group = blockIdx.x; group < ngroups_total; group += gridDim.x) {
        __syncthreads();
        const uint32_t t = find_tensor<GroupSpace>(desc, T, group);
        const TensorDesc d = desc[t];
        if (d.kind == kKindSmall || (ld_cg(&ws.sel[t].flags) & kSelFailed)) continue;
        const uint32_t Tkey = ld_cg(&ws.sel[t].T), m_eq = ld_cg(&ws.sel[t].m_eq);
        const uint32_t tile_in_t = (group - d.group0) * kWarps + warp;
        TileCands tc;
        tc.base = tc.cnt = tc.incl = tc.total = 0u;
        if (tile_in_t < d.ntiles) tc = load_tile_cands(cv, d.tile0 + tile_in_t, lane);
        uint32_t ngt, neq;
        group_tile_counts(cv, tc, Tkey, lane, ngt, neq);
        if (lane == 0) { sm.gt_tot[warp] = ngt; sm.eq_tot[warp] = neq; }
        if (EMIT) {
            // totals of the groups before this one in the tensor
            unsigned long long part = 0;
            for (uint32_t q = d.group0 + tid; q < group; q += kBlock) part += ld_cg(&cv.group_cnt[q]);
            part = warp_sum64(part);
            if (lane == 0) sm.red[warp] = part;
        }
        __syncthreads();
        scan_warp_totals(sm.gt_tot, sm.gt_ex, &sm.gt_sum, warp, lane);
        if (warp == 1) {
            uint32_t v = lane < kWarps ? sm.eq_tot[lane] : 0u;
            uint32_t inc = warp_incl_scan(v, lane);
            if (lane < kWarps) sm.eq_ex[lane] = inc - v;
            if (lane == 31) sm.eq_sum = inc;
        }
        if (EMIT && warp == 2) {
            unsigned long long v = lane < kWarps ? sm.red[lane] : 0ull;
            v = warp_sum64(v);
            if (lane == 0) sm.excl = v;
        }
        __syncthreads();
        if (!EMIT) {
            if (tid == 0)
                cv.group_cnt[group] = ((unsigned long long)sm.gt_sum << 31) | (unsigned long long)sm.eq_sum;
            continue;
        }
        uint32_t gpos = (uint32_t)(sm.excl >> 31) + sm.gt_ex[warp];
        uint32_t epos = (uint32_t)(sm.excl & 0x7FFFFFFFull) + sm.eq_ex[warp];
        for (uint32_t j0 = 0; j0 < tc.total; j0 += 32) {
            uint32_t j = j0 + lane;
            uint32_t slot = cand_slot(tc, j);
            float v = 0.f;
            uint32_t f = 0;
            if (j < tc.total) { const uint2 pr = ld_cg(&cv.pair[slot]); f = pr.x; v = __uint_as_float(pr.y); }
            uint32_t key = key_of(v);
            bool gt = j < tc.total && key > Tkey, eq = j < tc.total && key == Tkey;
            unsigned gb = __ballot_sync(0xFFFFFFFFu, gt), eb = __ballot_sync(0xFFFFFFFFu, eq);
            uint32_t mg = gpos + __popc(gb & lt_mask), me = epos + __popc(eb & lt_mask);
            if (gt || (eq && me < m_eq)) {
                uint32_t slot_out = mg + min(me, m_eq);
                if (slot_out < d.cap) {          // the residual already holds +0 for this entry
                    out_idx[d.out_off + slot_out] = f;
                    out_val[d.out_off + slot_out] = v;
                } else {
                    record_status(ws.hdr, -1 /*GC_E_INVALID*/, f);
                }
            } else if (j < tc.total) {
                r[f] = v;                        // candidate that is not sent: give its value back
            }
            gpos += __popc(gb); epos += __popc(eb);
        }
        if (out_count != nullptr && group == d.group0 && tid == 0) {
            out_count[t] = d.k;
            out_count[T + t] = d.k;
        }
    }
}

// ----------------------------------------------------------------------------- separate launches
static __global__ void __launch_bounds__(kBlock)
k_small_tensors(const TensorDesc* __restrict__ desc, uint32_t T, const uint32_t* __restrict__ small_ids,
                uint32_t n_small, const float* __restrict__ g, float* __restrict__ r,
                uint32_t* __restrict__ out_idx, float* __restrict__ out_val, uint32_t* __restrict__ out_count) {
    __shared__ BlockSmem sm;
    small_tensors_body(sm, desc, T, small_ids, n_small, g, r, out_idx, out_val, out_count);
}

static __global__ void __launch_bounds__(kBlock, 4)
k_fold_cand(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles,
            const float* __restrict__ g, float* __restrict__ r, WsView ws, CandView cv) {
    __shared__ BlockSmem sm;
    fold_cand_body(sm, desc, T, ntiles, g, r, ws, cv);
}

static __global__ void __launch_bounds__(kBlock)
k_cand_restore(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles, float* __restrict__ r,
               WsView ws, CandView cv) {
    cand_restore_body(desc, T, ntiles, r, ws, cv);
}

template <int LEVEL>
static __global__ void __launch_bounds__(kBlock)
k_cand_hist(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles, WsView ws, CandView cv) {
    __shared__ BlockSmem sm;
    if (ld_cg(&ws.hdr->overflow)) return;
    cand_hist_body<LEVEL>(sm, desc, T, ntiles, ws, cv);
}

template <bool EMIT>
static __global__ void __launch_bounds__(kBlock)
k_cand_compact(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ngroups_total,
               float* __restrict__ r, uint32_t* __restrict__ out_idx, float* __restrict__ out_val,
               uint32_t* __restrict__ out_count, WsView ws, CandView cv) {
    __shared__ BlockSmem sm;
    if (ld_cg(&ws.hdr->overflow)) return;
    cand_compact_body<EMIT>(sm, desc, T, ngroups_total, r, out_idx, out_val, out_count, ws, cv);
}

// ----------------------------------------------------------------------------- one launch
struct FusedArgs {
    const TensorDesc* desc;
    uint32_t T, ntiles, nstiles, ngroups;
    const uint32_t* small_ids;
    uint32_t n_small;
    const float* g;
    float* r;
    uint32_t* out_idx;
    float* out_val;
    uint32_t* out_count;
    WsView ws;               // main selection records, tile look-back words
    WsView sws;              // sample selection records
    WsView gws;              // records of the redo, gated by the main ones
    CandView cv;
};

// Whole top-k compress of one call in a single cooperative launch (one CTA per SM):
//   sample level 0 | sample level 1 | fold + candidates | candidate level 1 | candidate level 2
//   | group counts | emit, and -- only if a tensor's candidate set was too small or the list
//   overflowed -- the exact multi-pass redo of those tensors.
// Phases are separated by grid barriers; every decision taken after a barrier reads values
// that were final before it, so all CTAs take the same route.
static __global__ void __launch_bounds__(kBlock, 4)
k_compress_fused(const __grid_constant__ FusedArgs a) {
    __shared__ BlockSmem sm;
    uint32_t passed = 0, n_stamp = 0;
    WsHeader* hdr = a.ws.hdr;
    phase_stamp(hdr, n_stamp);
    // small tensors need nothing from anyone: run them first, no barrier of their own
    small_tensors_body(sm, a.desc, a.T, a.small_ids, a.n_small, a.g, a.r, a.out_idx, a.out_val, a.out_count);
    if (a.nstiles) {
        hist_body<0, SRC_SAMPLE>(sm, a.desc, a.T, a.nstiles, a.g, a.r, a.sws);
        if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
        hist_body<1, SRC_SAMPLE>(sm, a.desc, a.T, a.nstiles, a.g, a.r, a.sws);
        if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
    }
    fold_cand_body(sm, a.desc, a.T, a.ntiles, a.g, a.r, a.ws, a.cv);
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
    const bool overflow = ld_cg(&hdr->overflow) != 0u;
    if (!overflow) {
        cand_hist_body<1>(sm, a.desc, a.T, a.ntiles, a.ws, a.cv);
        if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
        cand_hist_body<2>(sm, a.desc, a.T, a.ntiles, a.ws, a.cv);
        if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
        cand_compact_body<false>(sm, a.desc, a.T, a.ngroups, a.r, a.out_idx, a.out_val, a.out_count, a.ws, a.cv);
        if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
        cand_compact_body<true>(sm, a.desc, a.T, a.ngroups, a.r, a.out_idx, a.out_val, a.out_count, a.ws, a.cv);
        __syncthreads();
        phase_stamp(hdr, n_stamp);
    }
    if (!overflow && ld_cg(&hdr->n_failed) == 0u) return;
    // redo (rare): first give the listed candidates of those tensors their values back, so that
    // r holds a for every element again
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
    cand_restore_body(a.desc, a.T, a.ntiles, a.r, a.ws, a.cv);
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
    hist_body<0, SRC_RESID>(sm, a.desc, a.T, a.ntiles, nullptr, a.r, a.gws);
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
    hist_body<1, SRC_RESID>(sm, a.desc, a.T, a.ntiles, nullptr, a.r, a.gws);
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
    hist_body<2, SRC_RESID>(sm, a.desc, a.T, a.ntiles, nullptr, a.r, a.gws);
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
    compact_body(sm, a.desc, a.T, a.ntiles, a.r, a.out_idx, a.out_val, a.out_count, a.gws, 0);
}

}  // namespace gc
