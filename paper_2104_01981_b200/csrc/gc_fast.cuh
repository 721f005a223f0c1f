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
#pragma once
#include "gc_kernels.cuh"

namespace gc {

struct CandView {
    uint2* pair;             // [cap] (flat index, bits of a = g + r) of each candidate
    uint2* chunk_info;       // [ntiles * kWarps] (first slot, count) per warp chunk
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
    if (lane < kWarps) info = cv.chunk_info[(size_t)tile * kWarps + lane];
    tc.base = info.x; tc.cnt = info.y;
    tc.incl = warp_incl_scan(tc.cnt, lane);
    tc.total = __shfl_sync(0xFFFFFFFFu, tc.incl, 31);
    return tc;
}
// slot of the j-th candidate of the tile (all lanes call; j >= total gives a harmless slot of chunk 0)
__device__ __forceinline__ uint32_t cand_slot(const TileCands& tc, uint32_t j) {
    uint32_t c = 0;
#pragma unroll
    for (int l = 0; l < kWarps; ++l) c += (j >= __shfl_sync(0xFFFFFFFFu, tc.incl, l)) ? 1u : 0u;
    c = min(c, (uint32_t)kWarps - 1u);
    uint32_t b = __shfl_sync(0xFFFFFFFFu, tc.base, c);
    uint32_t ex = __shfl_sync(0xFFFFFFFFu, tc.incl - tc.cnt, c);
    return b + (j - ex);
}

// ----------------------------------------------------------------------------- fold + candidates
// Asynchronous staging: each thread copies ITS OWN four 16-byte vectors of g and of r for the
// tiles ahead into shared memory with cp.async (no registers held, no barrier needed because a
// thread only ever reads back what it copied itself), kFoldStages tiles deep.  Tiles that touch
// the ragged first or last element of a tensor are loaded synchronously instead.
#ifndef GC_FOLD_ASYNC
#define GC_FOLD_ASYNC 1
#endif
#ifndef GC_FOLD_INTERLEAVE
#define GC_FOLD_INTERLEAVE 1
#endif
#ifndef GC_FOLD_MINBLOCKS
#define GC_FOLD_MINBLOCKS 1
#endif
constexpr int kFoldStages = GC_FOLD_ASYNC ? 3 : 0;
constexpr int kEmitStage = 64;              // candidates of one warp chunk staged in shared memory
constexpr size_t kFoldSmemBytes = (size_t)kFoldStages * 2 * kTile * sizeof(float);

__device__ __forceinline__ void cp_async16(void* smem, const void* gptr) {
    uint32_t sa = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(gptr) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ bool tile_is_interior(const TileGeom& q) {
    return q.lo == q.base && q.hi == q.base + (uint32_t)kTile;
}

// Reads g and r, writes a into r, emits candidates.  No block-wide barrier in the tile loop:
// every warp ranks and stores the candidates of its own chunk.
static __global__ void __launch_bounds__(kBlock, GC_FOLD_MINBLOCKS)
k_fold_cand(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles,
            const float* __restrict__ g, float* __restrict__ r, WsView ws, CandView cv) {
    constexpr int NB = 1 << level_bits(0);
    extern __shared__ __align__(16) unsigned char s_dyn[];
    float* const s_g = reinterpret_cast<float*>(s_dyn);
    float* const s_r = s_g + (size_t)kFoldStages * kTile;
    __shared__ uint32_t s_hist[NB];
    __shared__ uint32_t s_scratch[kWarps + 4];
    __shared__ uint32_t s_last;
    __shared__ uint2 s_emit[kWarps][kEmitStage];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#if GC_FOLD_INTERLEAVE
    // tile i of this CTA = blockIdx.x + i * gridDim.x: at any time the CTAs sweep one window
    const uint32_t tstep = gridDim.x;
    const uint32_t first = blockIdx.x;
    const uint32_t last = ntiles;
#else
    const uint32_t tstep = 1;
    const uint32_t per = (ntiles + gridDim.x - 1) / gridDim.x;
    const uint32_t first = blockIdx.x * per;
    const uint32_t last = min(ntiles, first + per);
#endif
    if (first >= last) return;
    for (int b = tid; b < NB; b += kBlock) s_hist[b] = 0u;
    __syncthreads();

    uint32_t t = find_tensor(desc, T, first);
    TensorDesc d = desc[t];
    uint32_t tau = d.sstride ? (cv.ssel[t].prefix << level_shift(1)) : 0u;
    uint32_t tiles_here = 0;
    uint32_t slab_next = 0, slab_left = 0;       // this warp's current slab (warp-uniform)

    // prefetch cursor
    uint32_t pt = t;
    TensorDesc pd = d;
    const uint32_t my_off = warp * kWarpChunk + lane * 4;        // + j * 128 elements
    auto issue = [&](uint32_t p, uint32_t seq) {
#if GC_FOLD_ASYNC
        if (p < last) {
            if (p >= pd.tile0 + pd.ntiles) { pt = find_tensor(desc, T, p); pd = desc[pt]; }
            const TileGeom q = tile_geom(pd, p - pd.tile0);
            if (tile_is_interior(q)) {
                const uint32_t st = seq % (uint32_t)kFoldStages;
                float* dg = s_g + (size_t)st * kTile + my_off;
                float* dr = s_r + (size_t)st * kTile + my_off;
                const float* gg = g + q.base + my_off;
                const float* gr = r + q.base + my_off;
#pragma unroll
                for (int j = 0; j < kVpt; ++j) {
                    cp_async16(dg + j * 128, gg + j * 128);
                    cp_async16(dr + j * 128, gr + j * 128);
                }
            }
        }
        cp_async_commit();
#endif
    };

    auto flush = [&]() {
        if (tiles_here == 0) return;
        __syncthreads();
        uint32_t* hist = ws.hist + (size_t)t * kHistBins;
        for (int b = tid; b < NB; b += kBlock) {
            uint32_t c = s_hist[b];
            if (c) { atomicAdd(hist + b, c); s_hist[b] = 0u; }
        }
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            uint32_t old = atomicAdd(&ws.sel[t].done[0], tiles_here);
            s_last = (old + tiles_here == d.ntiles) ? 1u : 0u;
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            select_step<0, true>(d.k, ws, t, s_scratch);
        }
        tiles_here = 0;
    };

#pragma unroll
    for (int s = 0; s < kFoldStages - 1; ++s) issue(first + s * tstep, s);

    uint32_t seq = 0;
    for (uint32_t tile = first; tile < last; tile += tstep, ++seq) {
        issue(tile + (kFoldStages - 1) * tstep, seq + kFoldStages - 1);
        if (tile >= d.tile0 + d.ntiles) {
            flush();
            t = find_tensor(desc, T, tile);
            d = desc[t];
            tau = d.sstride ? (cv.ssel[t].prefix << level_shift(1)) : 0u;
        }
        const TileGeom tg = tile_geom(d, tile - d.tile0);
        Tile tl;
#if GC_FOLD_ASYNC
        cp_async_wait<kFoldStages - 1>();
        if (tile_is_interior(tg)) {
            const uint32_t st = seq % (uint32_t)kFoldStages;
            const float* sgp = s_g + (size_t)st * kTile + my_off;
            const float* srp = s_r + (size_t)st * kTile + my_off;
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                const float4 gv = *reinterpret_cast<const float4*>(sgp + j * 128);
                const float4 rv = *reinterpret_cast<const float4*>(srp + j * 128);
                float4 a;
                a.x = __fadd_rn(gv.x, rv.x); a.y = __fadd_rn(gv.y, rv.y);
                a.z = __fadd_rn(gv.z, rv.z); a.w = __fadd_rn(gv.w, rv.w);
                *reinterpret_cast<float4*>(r + tg.base + my_off + j * 128) = a;
                tl.a[j][0] = a.x; tl.a[j][1] = a.y; tl.a[j][2] = a.z; tl.a[j][3] = a.w;
            }
            tl.valid = 0xFFFFu;
        } else
#endif
        {
            load_tile<true>(g, r, tg, warp, lane, tl);
        }
        uint32_t cnt[kVpt], cm = 0;
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
            cnt[j] = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                bool c = ((tl.valid >> (4 * j + e)) & 1u) && key_of(tl.a[j][e]) >= tau;
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
#ifndef GC_EXP_NO_CHUNKINFO
        if (lane == 0) cv.chunk_info[(size_t)tile * kWarps + warp] = make_uint2(cbase, fits ? wtot : 0u);
#endif
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
                            const uint2 pr = make_uint2(vec_index(tg.base, warp, lane, j) + e,
                                                        __float_as_uint(tl.a[j][e]));
                            if (staged) s_emit[warp][pos] = pr; else cv.pair[cbase + pos] = pr;
                            atomicAdd(&s_hist[key_of(tl.a[j][e]) >> level_shift(0)], 1u);
                            ++pos;
                        }
                    }
                }
            }
            if (staged) {
                __syncwarp();
                for (uint32_t i = lane; i < wtot; i += 32) cv.pair[cbase + i] = s_emit[warp][i];
                __syncwarp();
            }
        }
        ++tiles_here;
    }
#if GC_FOLD_ASYNC
    cp_async_wait<0>();
#endif
    flush();
}

// ----------------------------------------------------------------------------- candidate refinement
// Radix-select level 1 or 2 over the candidate lists.  CTAs take contiguous runs of tiles and
// walk them kWarps at a time, one warp per tile, always inside one tensor; counts go to a
// shared-memory histogram that is flushed when the tensor changes, and the CTA that completes
// a tensor's last tile runs the select step (same scheme as k_hist).
template <int LEVEL>
static __global__ void __launch_bounds__(kBlock)
k_cand_hist(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles, WsView ws, CandView cv) {
    constexpr int NB = 1 << level_bits(LEVEL);
    constexpr int SH = level_shift(LEVEL);
    __shared__ uint32_t s_hist[NB];
    __shared__ uint32_t s_scratch[kWarps + 4];
    __shared__ uint32_t s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (*(volatile uint32_t*)&ws.hdr->overflow) return;
    const uint32_t per = (ntiles + gridDim.x - 1) / gridDim.x;
    const uint32_t first = blockIdx.x * per;
    const uint32_t last = min(ntiles, first + per);
    if (first >= last) return;
    for (int b = tid; b < NB; b += kBlock) s_hist[b] = 0u;
    __syncthreads();

    uint32_t t = find_tensor(desc, T, first);
    TensorDesc d = desc[t];
    bool active = (ws.sel[t].flags & kSelFailed) == 0u;
    uint32_t prefix = ws.sel[t].prefix;
    uint32_t tiles_here = 0;

    auto flush = [&]() {
        if (!active || tiles_here == 0) { tiles_here = 0; return; }
        __syncthreads();
        uint32_t* hist = ws.hist + (size_t)t * kHistBins;
        for (int b = tid; b < NB; b += kBlock) {
            uint32_t c = s_hist[b];
            if (c) { atomicAdd(hist + b, c); s_hist[b] = 0u; }
        }
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            uint32_t old = atomicAdd(&ws.sel[t].done[LEVEL], tiles_here);
            s_last = (old + tiles_here == d.ntiles) ? 1u : 0u;
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            select_step<LEVEL, false>(0u, ws, t, s_scratch);
        }
        tiles_here = 0;
    };

    uint32_t batch = first;
    while (batch < last) {
        if (batch >= d.tile0 + d.ntiles) {
            flush();
            t = find_tensor(desc, T, batch);
            d = desc[t];
            active = (ws.sel[t].flags & kSelFailed) == 0u;
            prefix = ws.sel[t].prefix;
        }
        const uint32_t bend = min(min(last, d.tile0 + d.ntiles), batch + (uint32_t)kWarps);
        const uint32_t tile = batch + warp;
        if (active && tile < bend) {
            TileCands tc = load_tile_cands(cv, tile, lane);
            for (uint32_t j0 = 0; j0 < tc.total; j0 += 32) {
                uint32_t j = j0 + lane;
                uint32_t slot = cand_slot(tc, j);
                if (j < tc.total) {
                    uint32_t key = cv.pair[slot].y & kKeyMask;
                    if ((key >> (SH + level_bits(LEVEL))) == prefix)
                        atomicAdd(&s_hist[(key >> SH) & (NB - 1)], 1u);
                }
            }
        }
        tiles_here += bend - batch;
        batch = bend;
    }
    flush();
}

// ----------------------------------------------------------------------------- candidate compaction
// Index-ordered emission from the candidate lists.  A group is kWarps consecutive tiles of
// one tensor, one warp per tile; groups are handed out by ticket and exchange their
// (above-T, equal-T) counts through the look-back words, per tensor.  Sent entries are
// written to the output and zeroed in the residual (which already holds a).
static __global__ void __launch_bounds__(kBlock)
k_cand_compact(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ngroups_total,
               float* __restrict__ r, uint32_t* __restrict__ out_idx, float* __restrict__ out_val,
               uint32_t* __restrict__ out_count, WsView ws, CandView cv, int ticket_slot) {
    __shared__ uint32_t s_group;
    __shared__ uint32_t s_gt_tot[kWarps], s_eq_tot[kWarps], s_gt_ex[kWarps], s_eq_ex[kWarps];
    __shared__ uint32_t s_gt_sum, s_eq_sum;
    __shared__ unsigned long long s_excl;
    __shared__ int s_ok;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (*(volatile uint32_t*)&ws.hdr->overflow) return;
    const unsigned lt_mask = (1u << lane) - 1u;

    while (true) {
        __syncthreads();
        if (tid == 0) {
            uint32_t tk = atomicAdd(&ws.hdr->ticket[ticket_slot], 1u);
            if (*(volatile uint32_t*)&ws.hdr->abort) tk = 0xFFFFFFFFu;
            s_group = tk;
        }
        __syncthreads();
        const uint32_t group = s_group;
        if (group >= ngroups_total) break;
        const uint32_t t = find_tensor<GroupSpace>(desc, T, group);
        if (ws.sel[t].flags & kSelFailed) continue;
        const TensorDesc d = desc[t];
        const uint32_t Tkey = ws.sel[t].T, m_eq = ws.sel[t].m_eq;
        const uint32_t tile_in_t = (group - d.group0) * kWarps + warp;
        TileCands tc;
        tc.base = tc.cnt = tc.incl = tc.total = 0u;
        if (tile_in_t < d.ntiles) tc = load_tile_cands(cv, d.tile0 + tile_in_t, lane);

        // pass 1: counts of this warp's tile
        uint32_t ngt = 0, neq = 0;
        for (uint32_t j0 = 0; j0 < tc.total; j0 += 32) {
            uint32_t j = j0 + lane;
            uint32_t slot = cand_slot(tc, j);
            uint32_t key = j < tc.total ? (cv.pair[slot].y & kKeyMask) : 0u;
            bool gt = j < tc.total && key > Tkey, eq = j < tc.total && key == Tkey;
            ngt += __popc(__ballot_sync(0xFFFFFFFFu, gt));
            neq += __popc(__ballot_sync(0xFFFFFFFFu, eq));
        }
        if (lane == 0) { s_gt_tot[warp] = ngt; s_eq_tot[warp] = neq; }
        __syncthreads();
        scan_warp_totals(s_gt_tot, s_gt_ex, &s_gt_sum, warp, lane);
        if (warp == 1) {
            uint32_t v = lane < kWarps ? s_eq_tot[lane] : 0u;
            uint32_t inc = warp_incl_scan(v, lane);
            if (lane < kWarps) s_eq_ex[lane] = inc - v;
            if (lane == 31) s_eq_sum = inc;
        }
        __syncthreads();
        if (warp == 0) {
            unsigned long long agg = ((unsigned long long)s_gt_sum << 31) | (unsigned long long)s_eq_sum;
            bool ok;
            unsigned long long ex = lookback(ws.tile_state, group, d.group0, agg, lane, ws.hdr, ok);
            if (lane == 0) { s_excl = ex; s_ok = ok ? 1 : 0; }
        }
        __syncthreads();
        if (!s_ok) break;
        // pass 2: emit
        uint32_t gpos = (uint32_t)(s_excl >> 31) + s_gt_ex[warp];
        uint32_t epos = (uint32_t)(s_excl & 0x7FFFFFFFull) + s_eq_ex[warp];
        for (uint32_t j0 = 0; j0 < tc.total; j0 += 32) {
            uint32_t j = j0 + lane;
            uint32_t slot = cand_slot(tc, j);
            float v = 0.f;
            uint32_t f = 0;
            if (j < tc.total) { const uint2 pr = cv.pair[slot]; f = pr.x; v = __uint_as_float(pr.y); }
            uint32_t key = key_of(v);
            bool gt = j < tc.total && key > Tkey, eq = j < tc.total && key == Tkey;
            unsigned gb = __ballot_sync(0xFFFFFFFFu, gt), eb = __ballot_sync(0xFFFFFFFFu, eq);
            uint32_t mg = gpos + __popc(gb & lt_mask), me = epos + __popc(eb & lt_mask);
            if (gt || (eq && me < m_eq)) {
                uint32_t slot_out = mg + min(me, m_eq);
                if (slot_out < d.cap) {
                    out_idx[d.out_off + slot_out] = f;
                    out_val[d.out_off + slot_out] = v;
                    r[f] = 0.0f;
                } else {
                    record_status(ws.hdr, -1 /*GC_E_INVALID*/, f);
                }
            }
            gpos += __popc(gb); epos += __popc(eb);
        }
        if (out_count != nullptr && group == d.group0 && tid == 0) {
            out_count[t] = d.k;
            out_count[T + t] = d.k;
        }
    }
}

}  // namespace gc
