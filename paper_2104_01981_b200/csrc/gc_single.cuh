// Exact top-k of ONE large tensor in one cooperative launch with the candidates held in
// shared memory ("global top-k" workloads: the whole model is one flat tensor).
//
// Same idea as the general candidate path (sample -> fold + candidates -> radix select on the
// candidates -> index-ordered emission, exact multi-pass redo as the safety net), specialised:
//   * CTA b owns tiles b, b + G, b + 2G, ... (G = grid size): every CTA sees every region of
//     the tensor, so candidate counts stay balanced even when magnitudes differ between layers;
//   * a CTA appends the candidates of its own tiles to a private, contiguous region of the
//     candidate list (L2-resident) and keeps the per-chunk records in shared memory, so the
//     selection phases stream that region linearly with no indirection.  (Holding the
//     candidates themselves in shared memory was measured slower: the large carve-out leaves
//     too little L1 for the streaming loads of the fold pass.);
//   * each histogram level is flushed to global memory, and after the grid barrier EVERY CTA
//     scans it and derives the same prefix -- no completion counters, no designated CTA;
//   * output slots come from per-row totals: row i is the i-th tile of every CTA.
#pragma once
#include "gc_fast.cuh"

namespace gc {

struct SingleArgs {
    TensorDesc d;                    // the tensor (by value)
    const TensorDesc* desc;          // device table (for the redo phases)
    uint32_t ntiles, maxt, pool_cap; // tiles, max tiles per CTA, pool slots per CTA
    const float* g;
    float* r;
    uint32_t* out_idx;
    float* out_val;
    uint32_t* out_count;
    uint2* cand;                     // [gridDim.x * pool_cap] candidate list, one region per CTA
    uint32_t* hist5;                 // [5][kHistBins] sample L0, sample L1, candidates L0, L1, L2 (zeroed)
    unsigned long long* tile_cnt;    // [ntiles] (above-T << 31 | equal-T) per tile
    unsigned long long* row_tot;     // [maxt] the same summed over each row of tiles (zeroed)
    unsigned long long* seg_tot;     // [maxt][ceil(G/32)] ... and over each run of 32 CTAs of a row (zeroed)
    WsView ws, gws;
};

__device__ __forceinline__ void flush_hist(BlockSmem& sm, uint32_t* hist, int nb) {
    __syncthreads();
    for (int b = threadIdx.x; b < nb; b += kBlock) {
        uint32_t c = sm.hist[b];
        if (c) { atomicAdd(hist + b, c); sm.hist[b] = 0u; }
    }
}

static __global__ void __launch_bounds__(kBlock, 4)
k_topk_single(SingleArgs a) {
    __shared__ BlockSmem sm;
    __shared__ uint32_t s_used;
    extern __shared__ __align__(16) unsigned char s_dyn[];
    // dynamic shared memory: chunk records, chunk select counts, tile bases
    uint32_t* const rec = reinterpret_cast<uint32_t*>(s_dyn);                  // [maxt*kWarps] off<<10 | cnt
    uint32_t* const rec2 = rec + (size_t)a.maxt * kWarps;                      // [maxt*kWarps] gt<<16 | eq
    unsigned long long* const tile_base = reinterpret_cast<unsigned long long*>(rec2 + (size_t)a.maxt * kWarps);
    // This CTA's region.  Only this CTA (hence only this SM) ever writes or reads it, and it is
    // never read before it is written, so the later phases may read it through L1.
    uint2* const pool = a.cand + (size_t)blockIdx.x * a.pool_cap;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t G = gridDim.x, b = blockIdx.x;
    const TensorDesc& d = a.d;
    WsHeader* hdr = a.ws.hdr;
    uint32_t passed = 0;
    const uint32_t n_own = b < a.ntiles ? (a.ntiles - b + G - 1) / G : 0u;
    for (int i = tid; i < 2048; i += kBlock) sm.hist[i] = 0u;
    if (tid == 0) s_used = 0u;
    phase_stamp(hdr);

    // ---------------------------------------------------------------- sample (two radix levels)
    // One 4-element group out of d.sstride; a thread keeps the keys of its groups in registers
    // between the two levels.  tau_lo = the srank-th largest sampled key, cut to 21 bits.
    uint32_t tau = 0;
    {
        const uint32_t ngroups = (d.n + 3u) >> 2;
        const uint32_t nsg = (ngroups + d.sstride - 1) / d.sstride;
        constexpr int kMaxOwn = 2;                       // sample groups a thread may own
        uint32_t skey[kMaxOwn][4], sok = 0;
#pragma unroll
        for (int q = 0; q < kMaxOwn; ++q) {
            const uint64_t sg = (uint64_t)q * G * kBlock + (uint64_t)b * kBlock + tid;
            const uint64_t gi = sg * d.sstride;
            const bool in = sg < nsg && gi < ngroups;
            const uint32_t i0 = in ? (uint32_t)gi * 4u : 0u;
            float gv[4], rv[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool v = in && i0 + e < d.n;
                const uint32_t f = d.off + (v ? i0 + e : 0u);
                gv[e] = v ? __ldg(a.g + f) : 0.f;
                rv[e] = v ? ld_cg(a.r + f) : 0.f;
                sok |= (uint32_t)v << (4 * q + e);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) skey[q][e] = key_of(__fadd_rn(gv[e], rv[e]));
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kMaxOwn; ++q)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if ((sok >> (4 * q + e)) & 1u) atomicAdd(&sm.hist[skey[q][e] >> level_shift(0)], 1u);
        flush_hist(sm, a.hist5 + 0 * kHistBins, 1 << level_bits(0));
        if (!grid_barrier(hdr, passed, &sm.ok)) return;
        phase_stamp(hdr);
        uint32_t bin0, above0;
        const bool ok0 = block_select<(1 << level_bits(0)), false>(sm, a.hist5 + 0 * kHistBins, d.srank, bin0, above0);
        if (ok0) {
#pragma unroll
            for (int q = 0; q < kMaxOwn; ++q)
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (((sok >> (4 * q + e)) & 1u) && (skey[q][e] >> level_shift(0)) == bin0)
                        atomicAdd(&sm.hist[(skey[q][e] >> level_shift(1)) & ((1u << level_bits(1)) - 1u)], 1u);
        }
        flush_hist(sm, a.hist5 + 1 * kHistBins, 1 << level_bits(1));
        if (!grid_barrier(hdr, passed, &sm.ok)) return;
        phase_stamp(hdr);
        if (ok0) {
            uint32_t bin1, above1;
            if (block_select<(1 << level_bits(1)), false>(sm, a.hist5 + 1 * kHistBins, d.srank - above0, bin1, above1))
                tau = ((bin0 << level_bits(1)) | bin1) << level_shift(1);
        }
        // tau == 0 (sample too small for the rank): every element becomes a candidate, the pool
        // overflows and the exact redo takes over
    }

    // ---------------------------------------------------------------- fold + candidates
    const uint32_t my_off = warp * kWarpChunk + lane * 4;
    bool block_overflow = false;
    for (uint32_t i = 0; i < n_own; ++i) {
        const uint32_t tile = b + i * G;
        const TileGeom tg = tile_geom(d, tile);
        const bool interior = tg.lo == tg.base && tg.hi == tg.base + (uint32_t)kTile;
        float av[kVpt][4];
        uint32_t valid = 0xFFFFu;
        if (interior) {
            float4 gv[kVpt], rv[kVpt];
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                gv[j] = __ldg(reinterpret_cast<const float4*>(a.g + tg.base + my_off + j * 128));
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
                        v = __fadd_rn(__ldg(a.g + f), ld_cg(a.r + f));
                        valid |= 1u << (4 * j + e);
                    }
                    av[j][e] = v;
                }
            }
        }
        uint32_t cnt[kVpt], cm = 0;
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
            cnt[j] = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                bool c = key_of(av[j][e]) >= tau;
                if (!interior) c = c && ((valid >> (4 * j + e)) & 1u);
                cnt[j] += c;
                cm |= (uint32_t)c << (4 * j + e);
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
        const uint32_t zm = fits ? cm : 0u;
        if (interior) {
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                float4 o;
                o.x = ((zm >> (4 * j + 0)) & 1u) ? 0.0f : av[j][0];
                o.y = ((zm >> (4 * j + 1)) & 1u) ? 0.0f : av[j][1];
                o.z = ((zm >> (4 * j + 2)) & 1u) ? 0.0f : av[j][2];
                o.w = ((zm >> (4 * j + 3)) & 1u) ? 0.0f : av[j][3];
                *reinterpret_cast<float4*>(a.r + tg.base + my_off + j * 128) = o;
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
            if (zm != 0u) {
#pragma unroll
                for (int j = 0; j < kVpt; ++j) {
                    uint32_t pos = rk[j];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if ((zm >> (4 * j + e)) & 1u) {
                            const uint2 pr = make_uint2(tg.base + my_off + j * 128 + e, __float_as_uint(av[j][e]));
                            if (staged) sm.emit[warp][pos] = pr; else pool[off + pos] = pr;
                            atomicAdd(&sm.hist[key_of(av[j][e]) >> level_shift(0)], 1u);
                            ++pos;
                        }
                    }
                }
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
    flush_hist(sm, a.hist5 + 2 * kHistBins, 1 << level_bits(0));
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr);

    bool good = ld_cg(&hdr->overflow) == 0u;
    uint32_t Tkey = 0, m_eq = 0;
    if (good) {
        // ------------------------------------------------------------ radix select on the candidates
        uint32_t bin0, above0, bin1 = 0, above1 = 0, bin2 = 0, above2 = 0;
        good = block_select<(1 << level_bits(0)), false>(sm, a.hist5 + 2 * kHistBins, d.k, bin0, above0);
        if (good) {
            for (uint32_t i0 = tid; i0 < used; i0 += 4 * kBlock) {      // four loads in flight per thread
                uint32_t key[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t i = i0 + u * kBlock;
                    key[u] = i < used ? (pool[i].y & kKeyMask) : 0xFFFFFFFFu;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if ((key[u] >> level_shift(0)) == bin0)
                        atomicAdd(&sm.hist[(key[u] >> level_shift(1)) & ((1u << level_bits(1)) - 1u)], 1u);
            }
        }
        flush_hist(sm, a.hist5 + 3 * kHistBins, 1 << level_bits(1));
        if (!grid_barrier(hdr, passed, &sm.ok)) return;
        phase_stamp(hdr);
        if (good) good = block_select<(1 << level_bits(1)), false>(sm, a.hist5 + 3 * kHistBins, d.k - above0, bin1, above1);
        const uint32_t p1 = (bin0 << level_bits(1)) | bin1;
        if (good) {
            for (uint32_t i0 = tid; i0 < used; i0 += 4 * kBlock) {
                uint32_t key[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t i = i0 + u * kBlock;
                    key[u] = i < used ? (pool[i].y & kKeyMask) : 0xFFFFFFFFu;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if ((key[u] >> level_shift(1)) == p1) atomicAdd(&sm.hist[key[u] & ((1u << level_bits(2)) - 1u)], 1u);
            }
        }
        flush_hist(sm, a.hist5 + 4 * kHistBins, 1 << level_bits(2));
        if (!grid_barrier(hdr, passed, &sm.ok)) return;
        phase_stamp(hdr);
        if (good)
            good = block_select<(1 << level_bits(2)), false>(sm, a.hist5 + 4 * kHistBins, d.k - above0 - above1, bin2, above2);
        Tkey = (p1 << level_bits(2)) | bin2;
        m_eq = d.k - above0 - above1 - above2;
    }
    // `good` is the same in every CTA: it only depends on global histograms read after a barrier

    if (good) {
        // ------------------------------------------------------------ counts per chunk, tile, row, segment
        // (one thread per chunk here: a chunk holds a handful of candidates and there are
        // hundreds of chunks per CTA; the warp-per-tile form measured twice as slow)
        for (uint32_t c = tid; c < n_own * kWarps; c += kBlock) {
            const uint32_t rc = rec[c], off = rc >> 10, cnt = rc & 1023u;
            uint32_t ngt = 0, neq = 0;
            for (uint32_t j = 0; j < cnt; ++j) {
                const uint32_t key = pool[off + j].y & kKeyMask;
                ngt += key > Tkey; neq += key == Tkey;
            }
            rec2[c] = (ngt << 16) | neq;
        }
        __syncthreads();
        for (uint32_t i = tid; i < n_own; i += kBlock) {
            unsigned long long tot = 0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const uint32_t v = rec2[i * kWarps + w];
                tot += ((unsigned long long)(v >> 16) << 31) | (unsigned long long)(v & 0xFFFFu);
            }
            a.tile_cnt[b + i * G] = tot;
            atomicAdd(a.row_tot + i, tot);
            atomicAdd(a.seg_tot + (size_t)i * ((G + 31u) / 32u) + b / 32u, tot);
        }
        if (!grid_barrier(hdr, passed, &sm.ok)) return;
        phase_stamp(hdr);

        // ------------------------------------------------------------ slot of every own tile, emission
        // tile_base[i] = sum of the rows before row i + the tiles of row i owned by lower CTAs
        if (warp == 0) {
            unsigned long long run = 0;
            for (uint32_t i0 = 0; i0 < n_own; i0 += 32) {
                const uint32_t i = i0 + lane;
                const unsigned long long v = i < n_own ? ld_cg(a.row_tot + i) : 0ull;
                const unsigned long long inc = warp_incl_scan64(v, lane);
                if (i < n_own) tile_base[i] = run + inc - v;
                run += __shfl_sync(0xFFFFFFFFu, inc, 31);
            }
        }
        __syncthreads();
        const unsigned lt_mask = (1u << lane) - 1u;
        for (uint32_t i = warp; i < n_own; i += kWarps) {
            // tiles of row i owned by lower CTAs = whole 32-CTA segments below this CTA's segment
            // + the lower CTAs inside it: at most two loads per lane whatever b is
            const uint32_t nseg = (G + 31u) / 32u, myseg = b / 32u;
            unsigned long long part = 0;
            if ((uint32_t)lane < myseg) part += ld_cg(a.seg_tot + (size_t)i * nseg + lane);
            const uint32_t q = myseg * 32u + (uint32_t)lane;
            if (q < b) part += ld_cg(a.tile_cnt + (size_t)i * G + q);
            const unsigned long long base = tile_base[i] + warp_sum64(part);
            uint32_t gpos = (uint32_t)(base >> 31), epos = (uint32_t)(base & 0x7FFFFFFFull);
            const uint32_t rc = lane < kWarps ? rec[i * kWarps + lane] : 0u;
            const uint32_t cnt = rc & 1023u, off = rc >> 10;
            const uint32_t incl = warp_incl_scan(cnt, lane);
            const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 31);
            for (uint32_t j0 = 0; j0 < total; j0 += 32) {
                const uint32_t j = j0 + lane;
                uint32_t c = 0;
#pragma unroll
                for (int l = 0; l < kWarps; ++l) c += (j >= __shfl_sync(0xFFFFFFFFu, incl, l)) ? 1u : 0u;
                c = min(c, (uint32_t)kWarps - 1u);
                const uint32_t src = __shfl_sync(0xFFFFFFFFu, off, c) + (j - __shfl_sync(0xFFFFFFFFu, incl - cnt, c));
                const bool valid = j < total;
                uint2 pr = make_uint2(0u, 0u);
                if (valid) pr = pool[src];
                const uint32_t key = pr.y & kKeyMask;
                const bool gt = valid && key > Tkey, eq = valid && key == Tkey;
                const unsigned gb = __ballot_sync(0xFFFFFFFFu, gt), eb = __ballot_sync(0xFFFFFFFFu, eq);
                const uint32_t mg = gpos + __popc(gb & lt_mask), me = epos + __popc(eb & lt_mask);
                if (gt || (eq && me < m_eq)) {
                    const uint32_t slot = mg + min(me, m_eq);
                    if (slot < d.cap) {          // the residual already holds +0 for this entry
                        a.out_idx[d.out_off + slot] = pr.x;
                        a.out_val[d.out_off + slot] = __uint_as_float(pr.y);
                    } else {
                        record_status(hdr, -1 /*GC_E_INVALID*/, pr.x);
                    }
                } else if (valid) {
                    a.r[pr.x] = __uint_as_float(pr.y);   // candidate that is not sent: value goes back
                }
                gpos += __popc(gb); epos += __popc(eb);
            }
        }
        if (a.out_count != nullptr && b == 0 && tid == 0) { a.out_count[0] = d.k; a.out_count[1] = d.k; }
        __syncthreads();
        phase_stamp(hdr);
        exit_stamp(hdr);
        return;
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
    phase_stamp(hdr);
    hist_body<0, SRC_RESID>(sm, a.desc, 1u, a.ntiles, nullptr, a.r, a.gws);
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    hist_body<1, SRC_RESID>(sm, a.desc, 1u, a.ntiles, nullptr, a.r, a.gws);
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    hist_body<2, SRC_RESID>(sm, a.desc, 1u, a.ntiles, nullptr, a.r, a.gws);
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    compact_body(sm, a.desc, 1u, a.ntiles, a.r, a.out_idx, a.out_val, a.out_count, a.gws, 0);
}

}  // namespace gc
