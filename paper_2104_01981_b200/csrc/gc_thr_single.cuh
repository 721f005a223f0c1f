// Threshold-estimation variant for ONE large tensor in one cooperative launch.
//
//   sample   one 4-element group out of `sstride` is folded on the fly; its keys are kept (16 B
//            per group).  Coarse histogram (top 11 key bits, shared memory) + fine histogram
//            (top 18 bits, global atomics into scattered slots)          | grid barrier
//   level 2  every CTA derives the 18-bit prefix of the k_s-th largest sampled key, then puts the
//            kept keys under that prefix (a handful) on a short list and counts their low 13
//            bits in 8192 global bins                                    | grid barrier
//   fold     every CTA ranks the short list (or, if it overflowed, reads the 8192 bins):
//            tau = the EXACT k_s-th largest sampled key (it is part of the result's
//            definition, unlike the bracket of the top-k kernels).
//            a = g + r; every element with key >= tau is a hit: it goes to the CTA's region of
//            the hit list and leaves +0 in the residual.  Per-tile hit counts and 32-CTA
//            segment totals are published                                | grid barrier
//   emit     slot of a hit = hits in earlier tiles + hits before it in its tile (list order is
//            index order).  Hits whose slot reaches the capacity are not sent: their value
//            goes back into the residual and the call reports GC_W_TRUNCATED.
// If a CTA's region of the hit list overflows (far more hits than k), the listed values are
// restored and the ticket-ordered look-back pass redoes the emission with the same tau.
#pragma once
#include "gc_single.cuh"
#include "gc_threshold.cuh"

namespace gc {

struct ThrSingleArgs {
    TensorDesc d;                    // the tensor (by value)
    const TensorDesc* desc;          // device table (for the redo)
    uint32_t ntiles, maxt, pool_cap; // tiles, max tiles per CTA, hit slots per CTA
    uint32_t sample_rounds;          // sample groups per thread
    const float* g;
    float* r;
    uint32_t* out_idx;
    float* out_val;
    uint32_t* out_count;
    uint2* cand;                     // [gridDim.x * pool_cap] hit list, one region per CTA
    uint4* skeys;                    // [sample groups] the sampled keys
    uint32_t* hist5;                 // [0] coarse sample histogram, [1][0] short-list length (zeroed)
    uint32_t* hist13;                // [8192] low 13 bits of the sampled keys under the prefix (zeroed)
    uint2* mid;                      // [mid_cap] those keys (second word), as a short list
    uint32_t mid_cap;
    uint32_t* fine;                  // [kFineBins] fine sample histogram (zeroed)
    uint32_t* tile_cnt;              // [ntiles] hits per tile
    uint32_t* seg_tot;               // [maxt][ceil(G/32)] hits per run of 32 CTAs of a row (zeroed)
    WsView ws;
};

// (three CTAs per SM: 80 registers and no spills beat four at 64 registers, see k_topk_single)
static __global__ void __launch_bounds__(kBlock, 3)
k_threshold_single(const __grid_constant__ ThrSingleArgs a) {
    __shared__ BlockSmem sm;
    __shared__ uint32_t s_used;
    extern __shared__ __align__(16) unsigned char s_dyn[];
    uint32_t* const rec = reinterpret_cast<uint32_t*>(s_dyn);                  // [maxt*kWarps] off<<10 | cnt
    uint32_t* const rec2 = rec + (size_t)a.maxt * kWarps;                      // [maxt*kWarps] first slot of the chunk
    uint32_t* const tile_base = rec2 + (size_t)a.maxt * kWarps;                // [maxt]
    uint32_t* const row_sum = tile_base + a.maxt;                              // [maxt]
    uint2* const pool = a.cand + (size_t)blockIdx.x * a.pool_cap;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t G = gridDim.x, b = blockIdx.x;
    const TensorDesc& d = a.d;
    WsHeader* hdr = a.ws.hdr;
    uint32_t passed = 0, n_stamp = 0;
    const uint32_t n_own = b < a.ntiles ? (a.ntiles - b + G - 1) / G : 0u;
    const uint32_t nseg = (G + 31u) / 32u, myseg = b / 32u;
    for (int i = tid; i < 2048; i += kBlock) sm.hist[i] = 0u;
    if (tid == 0) s_used = 0u;
    phase_stamp(hdr, n_stamp);
    __syncthreads();

    // ---------------------------------------------------------------- sample, level 1
    const uint32_t ngroups = (d.n + 3u) >> 2;
    const uint32_t nsg = (ngroups + d.sstride - 1) / d.sstride;
    for (uint32_t q = 0; q < a.sample_rounds; ++q) {
        const uint64_t sg = (uint64_t)q * G * kBlock + (uint64_t)b * kBlock + tid;
        const bool mine = sg < nsg;                         // (every lane stays in the loop: the coarse counts are
        const uint64_t gi = sg * d.sstride;                 //  aggregated over the warp)  gi < ngroups by the definition of nsg
        const uint32_t i0 = mine ? (uint32_t)gi * 4u : 0u;
        float gv[4], rv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const bool v = mine && i0 + e < d.n;
            const uint32_t f = d.off + (v ? i0 + e : 0u);
            gv[e] = v ? __ldg(a.g + f) : 0.f;
            rv[e] = v ? ld_cg(a.r + f) : 0.f;
        }
        uint32_t key[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            key[e] = 0xFFFFFFFFu;                           // = not a sample
            if (mine && i0 + e < d.n) {
                key[e] = key_of(__fadd_rn(gv[e], rv[e]));
                atomicAdd(a.fine + fine_slot(key[e] >> kFineShift), 1u);
            }
            hist_add_warp(sm.hist, key[e] == 0xFFFFFFFFu ? 0xFFFFFFFFu : key[e] >> level_shift(0), lane);
        }
        if (mine) a.skeys[sg] = make_uint4(key[0], key[1], key[2], key[3]);
    }
    flush_hist(sm, a.hist5 + 0 * kHistBins, 1 << level_bits(0));
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);

    // ---------------------------------------------------------------- sample, level 2
    // prefix18 = top 18 bits of the k_s-th largest sampled key; rank18 = its rank inside that cell
    uint32_t prefix18 = 0xFFFFFFFFu, rank18 = 0;
    {
        const uint32_t want[1] = {d.srank};
        Picked pk[1];
        block_select_multi<(1 << level_bits(0)), 1>(sm, a.hist5 + 0 * kHistBins, want, pk);
        if (warp == 0) {
            uint32_t res = 0xFFFFFFFFu, rk = 0;
            if (pk[0].ok) {
                constexpr uint32_t PER = 1u << (kFineBits - 5);
                const uint32_t first = (pk[0].bin << kFineBits) + (1u << kFineBits) - 1u - (uint32_t)lane * PER;
                uint32_t v[PER], sum = 0;
#pragma unroll
                for (uint32_t j = 0; j < PER; ++j) { v[j] = ld_cg(a.fine + fine_slot(first - j)); sum += v[j]; }
                const uint32_t inc = warp_incl_scan(sum, lane);
                const uint32_t krem = d.srank - pk[0].above;
                uint32_t mine = 0xFFFFFFFFu, mrk = 0, run = inc - sum;
#pragma unroll
                for (uint32_t j = 0; j < PER; ++j) {
                    if (run < krem && krem <= run + v[j]) { mine = first - j; mrk = krem - run; }
                    run += v[j];
                }
                const unsigned hit = __ballot_sync(0xFFFFFFFFu, mine != 0xFFFFFFFFu);
                if (hit != 0u) {
                    res = __shfl_sync(0xFFFFFFFFu, mine, __ffs(hit) - 1);
                    rk = __shfl_sync(0xFFFFFFFFu, mrk, __ffs(hit) - 1);
                }
            }
            if (lane == 0) { sm.gt_tot[0] = res; sm.gt_tot[1] = rk; }
        }
        __syncthreads();
        prefix18 = sm.gt_tot[0]; rank18 = sm.gt_tot[1];
        __syncthreads();
    }
    // (prefix18 == ~0: the sample holds fewer than k_s keys -- cannot happen for a valid plan; tau
    // stays 0xFFFFFFFF then, nothing is a hit, and the counts say so)
    if (prefix18 != 0xFFFFFFFFu) {
        for (uint32_t q = 0; q < a.sample_rounds; ++q) {
            const uint64_t sg = (uint64_t)q * G * kBlock + (uint64_t)b * kBlock + tid;
            if (sg >= nsg) continue;
            const uint4 kv = a.skeys[sg];                    // written by this very thread
            const uint32_t kk[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if ((kk[e] >> kFineShift) == prefix18) {
                    atomicAdd(a.hist13 + (kk[e] & ((1u << kFineShift) - 1u)), 1u);
                    const uint32_t slot = atomicAdd(a.hist5 + kHistBins, 1u);      // short-list length
                    if (slot < a.mid_cap) a.mid[slot] = make_uint2(0u, kk[e]);
                }
        }
    }
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);

    // ---------------------------------------------------------------- exact tau, fold + hits
    uint32_t tau = 0xFFFFFFFFu;
    if (prefix18 != 0xFFFFFFFFu) {
        // The keys under the prefix are normally a few dozen: every CTA ranks that short list by
        // itself.  Only if it did not fit (thousands of sampled keys within 2^13 of each other)
        // are the 8192 bins read instead.
        const uint32_t m = ld_cg(a.hist5 + kHistBins);
        if (m <= a.mid_cap) {
            uint2 e[kMidRegs];
#pragma unroll
            for (uint32_t u = 0; u < kMidRegs; ++u)
                e[u] = u * kBlock + tid < m ? ld_cg(a.mid + u * kBlock + tid) : make_uint2(0u, 0u);
            uint32_t low, x0, x1;
            if (short_list_select(sm, e, a.mid, m, kFineShift, rank18,
                                  [&](const uint2& pr, uint32_t& v) { v = pr.y & ((1u << kFineShift) - 1u); return true; },
                                  low, x0, x1))
                tau = (prefix18 << kFineShift) | low;
        } else {
            const uint32_t want[1] = {rank18};
            Picked pk[1];
            block_select_multi<(1 << kFineShift), 1>(sm, a.hist13, want, pk);
            if (pk[0].ok) tau = (prefix18 << kFineShift) | pk[0].bin;
        }
    }
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
        const bool fits = off + wtot <= a.pool_cap && wtot < 1024u;
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
                __stcs(reinterpret_cast<float4*>(a.r + tg.base + my_off + j * 128), o);
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
    const uint32_t used = s_used;
    // hits per tile, per 32-CTA segment of a row
    for (uint32_t i = tid; i < n_own; i += kBlock) {
        uint32_t tot = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) tot += rec[i * kWarps + w] & 1023u;
        a.tile_cnt[b + i * G] = tot;
        atomicAdd(a.seg_tot + (size_t)i * nseg + myseg, tot);
    }
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);

    if (ld_cg(&hdr->overflow) == 0u) {
        // ------------------------------------------------------------ slots and emission
        for (uint32_t i0 = warp * 2u; i0 < n_own; i0 += kWarps * 2u) {
            uint32_t sv[2], tv[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const uint32_t i = i0 + u, q = myseg * 32u + (uint32_t)lane;
                sv[u] = (i < n_own && (uint32_t)lane < nseg) ? ld_cg(a.seg_tot + (size_t)i * nseg + lane) : 0u;
                tv[u] = (i < n_own && q < b) ? ld_cg(a.tile_cnt + (size_t)i * G + q) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const uint32_t row = __reduce_add_sync(0xFFFFFFFFu, sv[u]);
                const uint32_t low = __reduce_add_sync(0xFFFFFFFFu, tv[u] + ((uint32_t)lane < myseg ? sv[u] : 0u));
                if (lane == 0 && i0 + u < n_own) { row_sum[i0 + u] = row; tile_base[i0 + u] = low; }
            }
        }
        __syncthreads();
        if (warp == 0) {
            uint32_t run = 0;
            for (uint32_t i0 = 0; i0 < n_own; i0 += 32) {
                const uint32_t i = i0 + lane;
                const uint32_t v = i < n_own ? row_sum[i] : 0u;
                const uint32_t inc = warp_incl_scan(v, lane);
                if (i < n_own) tile_base[i] += run + inc - v;
                run += __shfl_sync(0xFFFFFFFFu, inc, 31);
            }
            // CTA 0 owns a tile in every row: its running total is the number of hits of the tensor
            if (b == 0 && lane == 0) {
                if (a.out_count != nullptr) { a.out_count[0] = min(run, d.cap); a.out_count[1] = run; }
                if (run > d.cap) record_status(hdr, 1 /*GC_W_TRUNCATED*/, 0);
            }
        }
        __syncthreads();
        for (uint32_t i = tid; i < n_own; i += kBlock) {
            uint32_t pos = tile_base[i];
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                rec2[i * kWarps + w] = pos;
                pos += rec[i * kWarps + w] & 1023u;
            }
        }
        __syncthreads();
        const uint32_t base0 = d.off & ~3u;
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
                const uint32_t rel = pr[u].x - base0;
                const uint32_t c = ((rel >> 12) / G) * kWarps + ((rel >> 9) & (kWarps - 1u));
                const uint32_t slot = rec2[c] + (i - (rec[c] >> 10));
                if (slot < d.cap) {
                    __stcs(a.out_idx + d.out_off + slot, pr[u].x);
                    __stcs(a.out_val + d.out_off + slot, __uint_as_float(pr[u].y));
                } else {
                    a.r[pr[u].x] = __uint_as_float(pr[u].y);        // beyond the capacity: stays in the residual
                }
            }
        }
        __syncthreads();
        phase_stamp(hdr, n_stamp);
        exit_stamp(hdr);
        return;
    }

    // ---------------------------------------------------------------- hit list overflowed (rare)
    // every listed hit gets its value back; the look-back pass then emits from r with the same tau
    for (uint32_t c = tid; c < n_own * kWarps; c += kBlock) {
        const uint32_t rc = rec[c], off = rc >> 10, cnt = rc & 1023u;
        for (uint32_t j = 0; j < cnt; ++j) {
            const uint2 pr = pool[off + j];
            a.r[pr.x] = __uint_as_float(pr.y);
        }
    }
    if (!grid_barrier(hdr, passed, &sm.ok)) return;
    phase_stamp(hdr, n_stamp);
    threshold_emit_body<false>(a.desc, 1u, a.ntiles, nullptr, a.r, a.out_idx, a.out_val, a.out_count, a.ws,
                               nullptr, tau, 0);
}

}  // namespace gc
