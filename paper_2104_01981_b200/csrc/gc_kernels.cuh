// Kernels of the exact multi-pass path: fold + radix-select histograms over the magnitude
// key, ordered compaction with residual zeroing, and the sparse decode.  Every kernel is a
// thin __global__ wrapper around a __device__ body so that the fused kernel can run the same
// bodies as phases of one launch.
#pragma once
#include <type_traits>

#include "gc_common.cuh"

namespace gc {

// ----------------------------------------------------------------------------- tile I/O
struct Tile {
    float a[kVpt][4];
    uint32_t valid;          // bit j*4+e set: element e of vector j belongs to this tile
};

// Loads the thread's vectors of one tile.  FOLD: a = g + r (one rounded fp32 add) and a is
// stored to r; otherwise a is read from r.  Interior vectors use 128-bit accesses; vectors
// that straddle the tensor's first or last element fall back to guarded scalar accesses.
// r is read at L2 (it may have been written by another CTA earlier in the same launch).
template <bool FOLD, typename GL = GradF32>
__device__ __forceinline__ void load_tile(const void* __restrict__ g, float* __restrict__ r,
                                          const TileGeom& tg, int warp, int lane, Tile& t) {
    t.valid = 0;
    float4 gv[kVpt], rv[kVpt];
    bool full[kVpt];
#pragma unroll
    for (int j = 0; j < kVpt; ++j) {
        uint32_t f0 = vec_index(tg.base, warp, lane, j);
        full[j] = (f0 >= tg.lo) && (f0 + 4 <= tg.hi);
        if (full[j]) {
            rv[j] = ld_cg(reinterpret_cast<const float4*>(r + f0));
            if (FOLD) gv[j] = GL::ld4(g, f0);
        }
    }
#pragma unroll
    for (int j = 0; j < kVpt; ++j) {
        uint32_t f0 = vec_index(tg.base, warp, lane, j);
        if (full[j]) {
            if (FOLD) {
                float4 s;
                s.x = __fadd_rn(gv[j].x, rv[j].x); s.y = __fadd_rn(gv[j].y, rv[j].y);
                s.z = __fadd_rn(gv[j].z, rv[j].z); s.w = __fadd_rn(gv[j].w, rv[j].w);
                *reinterpret_cast<float4*>(r + f0) = s;
                rv[j] = s;
            }
            t.a[j][0] = rv[j].x; t.a[j][1] = rv[j].y; t.a[j][2] = rv[j].z; t.a[j][3] = rv[j].w;
            t.valid |= 0xFu << (4 * j);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                uint32_t f = f0 + e;
                float v = 0.0f;
                if (f >= tg.lo && f < tg.hi) {
                    v = ld_cg(r + f);
                    if (FOLD) { v = __fadd_rn(GL::ld1(g, f), v); r[f] = v; }
                    t.valid |= 1u << (4 * j + e);
                }
                t.a[j][e] = v;
            }
        }
    }
}

// ----------------------------------------------------------------------------- block scans
// Exclusive scan of one value per warp (kWarps values) by warp 0; result in smem.
__device__ __forceinline__ void scan_warp_totals(uint32_t* s_tot, uint32_t* s_excl, uint32_t* s_sum,
                                                 int warp, int lane) {
    if (warp == 0) {
        uint32_t v = lane < kWarps ? s_tot[lane] : 0u;
        uint32_t inc = warp_incl_scan(v, lane);
        if (lane < kWarps) s_excl[lane] = inc - v;
        if (lane == 31) *s_sum = inc;
    }
}

// ----------------------------------------------------------------------------- select step
// Run by the CTA that completes the last tile of a tensor at one level: scans that tensor's
// histogram from the top bin down, finds the bin that holds the krem-th largest key, and
// clears the histogram for the next level.  `rank0` is the rank wanted at level 0.  With
// CHECK, a histogram holding fewer than krem keys marks the tensor as failed (the candidate
// set was too small) instead of selecting anything.
template <int LEVEL, bool CHECK>
__device__ void select_step(uint32_t rank0, const WsView& ws, uint32_t t,
                            uint32_t* s_scratch /* >= kWarps + 4 words */) {
    constexpr int NB = 1 << level_bits(LEVEL);
    constexpr int BPT = (NB + kBlock - 1) / kBlock;          // bins per thread
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t* hist = ws.hist + (size_t)t * kHistBins;
    TensorSel* sel = ws.sel + t;
    const uint32_t krem = level_is_first(LEVEL) ? rank0 : ld_cg(&sel->krem);
    const uint32_t prefix = level_is_first(LEVEL) ? 0u : ld_cg(&sel->prefix);
    // thread `tid` owns BPT consecutive bins, counted from the largest key downwards
    uint32_t c[BPT];
    uint32_t sum = 0;
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        int b = NB - 1 - (tid * BPT + i);
        c[i] = (b >= 0) ? ld_cg(hist + b) : 0u;
        if (b >= 0) hist[b] = 0u;
        sum += c[i];
    }
    uint32_t inc = warp_incl_scan(sum, lane);
    if (lane == 31) s_scratch[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        uint32_t v = lane < kWarps ? s_scratch[lane] : 0u;
        uint32_t wi = warp_incl_scan(v, lane);
        if (lane < kWarps) s_scratch[lane] = wi - v;
        if (lane == kWarps - 1) s_scratch[kWarps] = wi;      // total keys in the histogram
    }
    __syncthreads();
    if (CHECK && s_scratch[kWarps] < krem) {
        if (tid == 0) {
            sel->flags = kSelFailed;
            atomicAdd(&ws.hdr->n_failed, 1u);
        }
        __syncthreads();
        return;
    }
    uint32_t above = s_scratch[warp] + inc - sum;            // keys in bins above this thread's
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        int b = NB - 1 - (tid * BPT + i);
        if (b >= 0 && above < krem && krem <= above + c[i]) {
            uint32_t np = (prefix << level_bits(LEVEL)) | (uint32_t)b;
            sel->prefix = np;
            sel->krem = krem - above;
            if (LEVEL == kLevels - 1) { sel->T = np; sel->m_eq = krem - above; }
        }
        above += c[i];
    }
    __syncthreads();
}

// Shared tail of every histogram phase: add the CTA's shared-memory histogram of tensor t to
// the global one, count the tiles it covered, and let the CTA that completes the tensor run
// the select step.
template <int LEVEL, bool CHECK>
__device__ __forceinline__ void flush_and_select(BlockSmem& sm, const WsView& ws, uint32_t t,
                                                 uint32_t tiles_here, uint32_t tiles_of_tensor,
                                                 uint32_t rank0) {
    constexpr int NB = 1 << level_bits(LEVEL);
    const int tid = threadIdx.x;
    __syncthreads();
    uint32_t* hist = ws.hist + (size_t)t * kHistBins;
    for (int b = tid; b < NB; b += kBlock) {
        uint32_t c = sm.hist[b];
        if (c) { atomicAdd(hist + b, c); sm.hist[b] = 0u; }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        uint32_t old = atomicAdd(&ws.sel[t].done[LEVEL], tiles_here);
        sm.last = (old + tiles_here == tiles_of_tensor) ? 1u : 0u;
    }
    __syncthreads();
    if (sm.last) {
        __threadfence();
        select_step<LEVEL, CHECK>(rank0, ws, t, sm.scratch);
    }
}

// ----------------------------------------------------------------------------- CTA-wide select
// Every thread of the CTA: find the bin of `hist` (NB bins; in global memory and complete, or in
// this CTA's shared memory) that holds the krem-th largest key.  Returns false if the histogram
// holds fewer than krem keys.  All threads get the same result.
template <int NB, bool IN_SMEM>
__device__ bool block_select(BlockSmem& sm, const uint32_t* hist, uint32_t krem, uint32_t& bin,
                             uint32_t& above_out) {
    constexpr int BPT = (NB + kBlock - 1) / kBlock;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t c[BPT], sum = 0;
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        int b = NB - 1 - (tid * BPT + i);
        c[i] = (b >= 0) ? (IN_SMEM ? hist[b] : ld_cg(hist + b)) : 0u;
        sum += c[i];
    }
    uint32_t inc = warp_incl_scan(sum, lane);
    __syncthreads();
    if (lane == 31) sm.scratch[warp] = inc;
    if (tid == 0) { sm.gt_sum = 0xFFFFFFFFu; sm.eq_sum = 0u; }
    __syncthreads();
    if (warp == 0) {
        uint32_t v = lane < kWarps ? sm.scratch[lane] : 0u;
        uint32_t wi = warp_incl_scan(v, lane);
        if (lane < kWarps) sm.scratch[lane] = wi - v;
        if (lane == kWarps - 1) sm.scratch[kWarps] = wi;
    }
    __syncthreads();
    uint32_t above = sm.scratch[warp] + inc - sum;
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        int b = NB - 1 - (tid * BPT + i);
        if (b >= 0 && above < krem && krem <= above + c[i]) { sm.gt_sum = (uint32_t)b; sm.eq_sum = above; }
        above += c[i];
    }
    __syncthreads();
    bin = sm.gt_sum; above_out = sm.eq_sum;
    const bool ok = sm.scratch[kWarps] >= krem && bin != 0xFFFFFFFFu;
    __syncthreads();
    return ok;
}

// Zeroes n16 16-byte words (the control block of a workspace).
static __global__ void __launch_bounds__(kBlock) k_clear(uint4* __restrict__ p, size_t n16) {
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    for (size_t i = (size_t)blockIdx.x * kBlock + threadIdx.x; i < n16; i += (size_t)gridDim.x * kBlock) p[i] = z;
}

// The same for several workspaces at once (blockIdx.y picks the workspace).
struct ClearMany { uint4* p[12]; };
static __global__ void __launch_bounds__(kBlock) k_clear_many(const __grid_constant__ ClearMany c, size_t n16) {
    uint4* const p = c.p[blockIdx.y];
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    for (size_t i = (size_t)blockIdx.x * kBlock + threadIdx.x; i < n16; i += (size_t)gridDim.x * kBlock) p[i] = z;
}

// ----------------------------------------------------------------------------- histogram pass
// One radix-select level over all tensors.  CTAs take contiguous runs of tiles, keep a
// shared-memory histogram while the tensor stays the same, flush it with global atomics when
// it changes, and the CTA that completes a tensor's last tile runs the select step.
//   SRC_FOLD   (level 0): reads g and r, writes a = g + r into r (12 bytes per element)
//   SRC_RESID:            reads a from r (4 bytes per element)
//   SRC_SAMPLE:           walks the tensor's sample (one 4-element group out of `sstride`),
//                         a = g + r is computed but not stored; rank = the tensor's srank
// At levels above 0 only keys under the prefix fixed so far are counted.
constexpr int SRC_FOLD = 0, SRC_RESID = 1, SRC_SAMPLE = 2;

template <int LEVEL, int SRC>
__device__ void hist_body(BlockSmem& sm, const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles,
                          const float* __restrict__ g, float* __restrict__ r, const WsView& ws,
                          uint32_t G, uint32_t b_in_group) {       // G CTAs share the work, this is CTA b of them
    using S = typename std::conditional<SRC == SRC_SAMPLE, SampleSpace, FullSpace>::type;
    constexpr int NB = 1 << level_bits(LEVEL);
    constexpr int SH = level_shift(LEVEL);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (nothing_to_redo(ws)) return;
    const uint32_t per = (ntiles + G - 1) / G;
    const uint32_t first = b_in_group * per;
    const uint32_t last = min(ntiles, first + per);
    if (first >= last) return;
    for (int b = tid; b < NB; b += kBlock) sm.hist[b] = 0u;
    __syncthreads();

    uint32_t t = find_tensor<S>(desc, T, first);
    TensorDesc d = desc[t];
    bool active = gate_open(ws, t, d);
    uint32_t prefix = level_is_first(LEVEL) ? 0u : ld_cg(&ws.sel[t].prefix);
    uint32_t tiles_here = 0;

    for (uint32_t tile = first; tile < last; ++tile) {
        if (tile >= S::tile0(d) + S::ntiles(d)) {
            if (active && tiles_here)
                flush_and_select<LEVEL, false>(sm, ws, t, tiles_here, S::ntiles(d), S::rank(d));
            tiles_here = 0;
            t = find_tensor<S>(desc, T, tile);
            d = desc[t];
            active = gate_open(ws, t, d);
            prefix = level_is_first(LEVEL) ? 0u : ld_cg(&ws.sel[t].prefix);
        }
        if (!active) continue;
        if (SRC == SRC_SAMPLE) {
            // sample tile: kSampleTile sample groups, one per thread; all loads are issued
            // before any of them is used
            const uint32_t ngroups = (d.n + 3u) >> 2;
            const uint64_t gi = (uint64_t)((tile - d.stile0) * (uint32_t)kSampleTile + tid) * d.sstride;
            const uint32_t i0 = (uint32_t)min(gi, (uint64_t)ngroups) * 4u;
            float gv[4], rv[4];
            uint32_t ok = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                bool v = gi < ngroups && i0 + e < d.n;
                uint32_t f = d.off + (v ? i0 + e : 0u);
                gv[e] = v ? __ldg(g + f) : 0.f;
                rv[e] = v ? ld_cg(r + f) : 0.f;
                ok |= (uint32_t)v << e;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                uint32_t key = key_of(__fadd_rn(gv[e], rv[e]));
                bool in = (ok >> e) & 1u;
                if (!level_is_first(LEVEL)) in = in && ((key >> (SH + level_bits(LEVEL))) == prefix);
                if (in) atomicAdd(&sm.hist[(key >> SH) & (NB - 1)], 1u);
            }
        } else {
            TileGeom tg = tile_geom(d, tile - d.tile0);
            Tile tl;
            load_tile<SRC == SRC_FOLD>(g, r, tg, warp, lane, tl);
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    uint32_t key = key_of(tl.a[j][e]);
                    bool in = (tl.valid >> (4 * j + e)) & 1u;
                    if (!level_is_first(LEVEL)) in = in && ((key >> (SH + level_bits(LEVEL))) == prefix);
                    if (in) atomicAdd(&sm.hist[(key >> SH) & (NB - 1)], 1u);
                }
            }
        }
        ++tiles_here;
    }
    if (active && tiles_here) flush_and_select<LEVEL, false>(sm, ws, t, tiles_here, S::ntiles(d), S::rank(d));
}

template <int LEVEL, int SRC>
__device__ __forceinline__ void hist_body(BlockSmem& sm, const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles,
                                          const float* __restrict__ g, float* __restrict__ r, const WsView& ws) {
    hist_body<LEVEL, SRC>(sm, desc, T, ntiles, g, r, ws, gridDim.x, blockIdx.x);
}

template <int LEVEL, int SRC>
__global__ void __launch_bounds__(kBlock)
k_hist(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles,
       const float* __restrict__ g, float* __restrict__ r, WsView ws) {
    __shared__ BlockSmem sm;
    hist_body<LEVEL, SRC>(sm, desc, T, ntiles, g, r, ws);
}

// ----------------------------------------------------------------------------- compaction
// Ordered emission of the selected entries.  Tiles are handed out by an atomic ticket so
// that every predecessor of a running tile is itself running or finished; the exclusive
// counts (keys above T, keys equal to T) of a tile within its tensor come from the look-back
// exchange.  An element is sent iff key > T, or key == T and fewer than m_eq equal keys
// precede it in the tensor.  Sent elements are written as (flat index, value) at their rank
// and zeroed in the residual.
static __device__ __noinline__ void compact_body(BlockSmem& sm, const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles,
                             float* __restrict__ r, uint32_t* __restrict__ out_idx,
                             float* __restrict__ out_val, uint32_t* __restrict__ out_count,
                             const WsView& ws, int ticket_slot) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (nothing_to_redo(ws)) return;

    while (true) {
        __syncthreads();
        if (tid == 0) {
            uint32_t tk = atomicAdd(&ws.hdr->ticket[ticket_slot], 1u);
            if (ld_cg(&ws.hdr->abort)) tk = 0xFFFFFFFFu;
            sm.tile = tk;
        }
        __syncthreads();
        const uint32_t tile = sm.tile;
        if (tile >= ntiles) break;
        const uint32_t t = find_tensor(desc, T, tile);
        const TensorDesc d = desc[t];
        if (!gate_open(ws, t, d)) continue;
        const uint32_t Tkey = ld_cg(&ws.sel[t].T), m_eq = ld_cg(&ws.sel[t].m_eq);
        const TileGeom tg = tile_geom(d, tile - d.tile0);
        Tile tl;
        load_tile<false>(nullptr, r, tg, warp, lane, tl);

        uint32_t cg[kVpt], ce[kVpt], gtm = 0, eqm = 0;
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
            cg[j] = 0; ce[j] = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                uint32_t key = key_of(tl.a[j][e]);
                bool v = (tl.valid >> (4 * j + e)) & 1u;
                bool gt = v && key > Tkey, eq = v && key == Tkey;
                cg[j] += gt; ce[j] += eq;
                gtm |= (uint32_t)gt << (4 * j + e);
                eqm |= (uint32_t)eq << (4 * j + e);
            }
        }
        uint32_t rg[kVpt], re[kVpt], wg, we;
        warp_rank(cg, lane, rg, wg);
        warp_rank(ce, lane, re, we);
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
        if (warp == 0) {
            unsigned long long agg = ((unsigned long long)sm.gt_sum << 31) | (unsigned long long)sm.eq_sum;
            bool ok;
            unsigned long long ex = lookback(ws.tile_state, tile, d.tile0, agg, lane, ws.hdr, ok);
            if (lane == 0) { sm.excl = ex; sm.ok = ok ? 1 : 0; }
        }
        __syncthreads();
        if (!sm.ok) break;
        const uint32_t gt_before = (uint32_t)(sm.excl >> 31) + sm.gt_ex[warp];
        const uint32_t eq_before = (uint32_t)(sm.excl & 0x7FFFFFFFull) + sm.eq_ex[warp];
        if ((gtm | eqm) != 0u) {
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                uint32_t gpos = gt_before + rg[j], epos = eq_before + re[j];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    bool gt = (gtm >> (4 * j + e)) & 1u, eq = (eqm >> (4 * j + e)) & 1u;
                    if (gt || (eq && epos < m_eq)) {
                        uint32_t slot = gpos + min(epos, m_eq);
                        uint32_t f = vec_index(tg.base, warp, lane, j) + e;
                        if (slot < d.cap) {
                            uint32_t pos = d.out_off + slot;
                            out_idx[pos] = f;
                            out_val[pos] = tl.a[j][e];
                            r[f] = 0.0f;
                        } else {      // cannot happen with a correct select; never write outside
                            record_status(ws.hdr, -1 /*GC_E_INVALID*/, f);
                        }
                    }
                    gpos += gt; epos += eq;
                }
            }
        }
        if (out_count != nullptr && tile == d.tile0 && tid == 0) {
            out_count[t] = d.k;
            out_count[T + t] = d.k;
        }
    }
}

static __global__ void __launch_bounds__(kBlock)
k_compact(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles,
          float* __restrict__ r, uint32_t* __restrict__ out_idx, float* __restrict__ out_val,
          uint32_t* __restrict__ out_count, WsView ws, int ticket_slot) {
    __shared__ BlockSmem sm;
    compact_body(sm, desc, T, ntiles, r, out_idx, out_val, out_count, ws, ticket_slot);
}

// ----------------------------------------------------------------------------- decode
// One sparse set added into the dense buffer.  Indices of one set are distinct, so plain
// read-modify-write is race free; sets are applied by consecutive launches in worker order,
// which fixes the order of the fp32 additions per element.
static __global__ void __launch_bounds__(256)
k_scatter_add(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t total_cap, uint32_t total_n,
              const uint32_t* __restrict__ idx, const float* __restrict__ val,
              const uint32_t* __restrict__ count, float* __restrict__ out, WsHeader* hdr) {
    uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= total_cap) return;
    if (count != nullptr) {
        // slot j belongs to the last tensor whose out_off <= j; it is live iff below the count
        uint32_t lo = 0, hi = T;
        while (hi - lo > 1) {
            uint32_t mid = (lo + hi) >> 1;
            if (__ldg(&desc[mid].out_off) <= j) lo = mid; else hi = mid;
        }
        if (j - __ldg(&desc[lo].out_off) >= __ldg(count + lo)) return;
    }
    uint32_t i = __ldg(idx + j);
    if (i >= total_n) { record_status(hdr, -1 /*GC_E_INVALID*/, j); return; }
    out[i] = __fadd_rn(out[i], __ldg(val + j));
}

}  // namespace gc
