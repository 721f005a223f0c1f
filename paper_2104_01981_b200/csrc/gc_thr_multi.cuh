// Threshold-estimation variant for MANY tensors in one cooperative launch.
//
//   sample   per tensor: coarse histogram (top 11 key bits) of the strided sample, the sampled
//            keys are kept.  Tensors that fit one tile are finished here by one CTA each,
//            between the arrival at and the wait on the barrier       | grid barrier
//   tau      one CTA per remaining tensor: coarse bin from the histogram, then two more radix
//            levels over that tensor's kept keys in shared memory: the EXACT k_s-th largest
//            sampled key (it is part of the result's definition)      | grid barrier
//   fold     CTA b walks its contiguous run of tiles, segment by segment (a segment = one
//            tensor's tiles inside the run): a = g + r, every element with key >= tau is a hit,
//            goes to the CTA's region of the hit list and leaves +0 in the residual; per-tile
//            hit counts are published                                  | grid barrier
//   emit     slot of a hit = hits of the tensor's earlier tiles + hits before it in its tile;
//            hits whose slot reaches the tensor's capacity get their value written back.
// A full hit-list region restores the listed values and hands over to the ticket-ordered
// look-back pass with the same thresholds.
#pragma once
#include "gc_multi.cuh"
#include "gc_threshold.cuh"

namespace gc {

struct ThrMultiArgs {
    const TensorDesc* desc;
    uint32_t T, ntiles, nstiles;
    uint32_t per;                    // tiles per CTA (contiguous run)
    uint32_t pool_cap;               // hit slots per CTA
    uint32_t ntab;                   // T if the tile tables fit in shared memory, else 0
    const uint32_t* small_ids;       // tensors that fit one tile
    uint32_t n_small;
    const uint32_t* reg_ids;         // the others (with elements)
    uint32_t n_reg;
    const float* g;
    float* r;
    uint32_t* out_idx;
    float* out_val;
    uint32_t* out_count;
    uint2* cand;                     // [gridDim.x * pool_cap]
    uint32_t* shist;                 // [T][kHistBins] coarse sample histogram (zeroed)
    uint4* skeys;                    // [nstiles * kBlock] the sampled keys
    uint32_t* tile_cnt;              // [ntiles] hits per tile
    TensorSel* tsel;                 // [T] .T receives tau
    WsView ws;
};

// A tensor that fits one tile, start to finish by one CTA: exact k_s-th largest key of its own
// sample (three shared-memory radix levels over registers), then every element at or above it
// in index order, up to the capacity.
static __device__ __noinline__ void small_threshold_body(BlockSmem& sm, const TensorDesc& d, uint32_t t, uint32_t T,
                                                         const float* __restrict__ g, float* __restrict__ r,
                                                         uint32_t* __restrict__ out_idx, float* __restrict__ out_val,
                                                         uint32_t* __restrict__ out_count, WsHeader* hdr) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const TileGeom tg = tile_geom(d, 0u);
    Tile tl;
    load_tile<true>(g, r, tg, warp, lane, tl);           // r = a = g + r; sent entries get +0 below
    // sample membership: one 4-element group of the TENSOR (not of the flat buffer) out of sstride
    uint32_t smask = 0;
#pragma unroll
    for (int j = 0; j < kVpt; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint32_t f = vec_index(tg.base, warp, lane, j) + e;
            if (((tl.valid >> (4 * j + e)) & 1u) && (((f - d.off) >> 2) % d.sstride) == 0u) smask |= 1u << (4 * j + e);
        }
    uint32_t prefix = 0, krem = d.srank;
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
                bool in = (smask >> (4 * j + e)) & 1u;
                if (level > 0) in = in && ((key >> (sh + bits)) == prefix);
                if (in) atomicAdd(&sm.hist[(key >> sh) & ((1u << bits) - 1u)], 1u);
            }
        }
        __syncthreads();
        uint32_t bin, above;
        if (level == 0) block_select<(1 << level_bits(0)), true>(sm, sm.hist, krem, bin, above);
        else block_select<(1 << level_bits(1)), true>(sm, sm.hist, krem, bin, above);
        prefix = (prefix << bits) | bin;
        krem -= above;
    }
    const uint32_t tau = prefix;
    uint32_t cnt[kVpt], hm = 0;
#pragma unroll
    for (int j = 0; j < kVpt; ++j) {
        cnt[j] = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const bool h = ((tl.valid >> (4 * j + e)) & 1u) && key_of(tl.a[j][e]) >= tau;
            cnt[j] += h;
            hm |= (uint32_t)h << (4 * j + e);
        }
    }
    uint32_t rk[kVpt], wtot;
    warp_rank(cnt, lane, rk, wtot);
    __syncthreads();
    if (lane == 0) sm.gt_tot[warp] = wtot;
    __syncthreads();
    scan_warp_totals(sm.gt_tot, sm.gt_ex, &sm.gt_sum, warp, lane);
    __syncthreads();
    if (hm != 0u) {
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
            uint32_t slot = sm.gt_ex[warp] + rk[j];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if ((hm >> (4 * j + e)) & 1u) {
                    if (slot < d.cap) {
                        const uint32_t f = vec_index(tg.base, warp, lane, j) + e;
                        out_idx[d.out_off + slot] = f;
                        out_val[d.out_off + slot] = tl.a[j][e];
                        r[f] = 0.0f;
                    }
                    ++slot;
                }
            }
        }
    }
    if (tid == 0) {
        const uint32_t hits = sm.gt_sum;
        if (out_count != nullptr) { out_count[t] = min(hits, d.cap); out_count[T + t] = hits; }
        if (hits > d.cap) record_status(hdr, 1 /*GC_W_TRUNCATED*/, t);
    }
    __syncthreads();
}

// The whole threshold compress of one worker by the G CTAs of one group (this CTA is number b of
// them); the group's barriers count on the worker's own workspace header.
static __device__ __forceinline__ void threshold_multi_body(const ThrMultiArgs& a, const uint32_t G, const uint32_t b,
                                                            BlockSmem& sm, uint32_t& s_used, uint32_t& s_cnt,
                                                            unsigned char* s_dyn) {
    uint32_t* const rec = reinterpret_cast<uint32_t*>(s_dyn);                  // [per*kWarps] off<<10 | cnt
    uint32_t* const rec2 = rec + (size_t)a.per * kWarps;                       // [per*kWarps] first slot of the chunk
    uint32_t* const seg = rec2 + (size_t)a.per * kWarps;                       // [per][kSegWords]
    uint32_t* const tab_tile0 = seg + (size_t)a.per * kSegWords;               // [ntab] first tile of every tensor
    uint32_t* const tab_stile0 = tab_tile0 + a.ntab;                           // [ntab] first sample tile
    uint2* const pool = a.cand + (size_t)b * a.pool_cap;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    WsHeader* hdr = a.ws.hdr;
    uint32_t passed = 0, n_stamp = 0;
    const uint32_t first = min(a.ntiles, b * a.per), last = min(a.ntiles, first + a.per);
    const uint32_t ntl = last - first;
    for (int i = tid; i < 2048; i += kBlock) sm.hist[i] = 0u;
    for (uint32_t i = tid; i < ntl * kWarps; i += kBlock) { rec[i] = 0u; rec2[i] = 0u; }
    if (tid == 0) { s_used = 0u; s_cnt = 0u; }
    for (uint32_t t = tid; t < a.ntab; t += kBlock) {
        tab_tile0[t] = a.desc[t].tile0;
        tab_stile0[t] = a.desc[t].stile0;
    }
    phase_stamp(hdr, n_stamp, b);
    __syncthreads();
    auto owner = [&](const uint32_t* tab, uint32_t tile) -> uint32_t {    // last t with tab[t] <= tile
        uint32_t lo = 0, hi = a.ntab;
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (tab[mid] <= tile) lo = mid; else hi = mid;
        }
        return lo;
    };

    // ---------------------------------------------------------------- sample: coarse histogram, keys kept
    if (a.nstiles) {
        const uint32_t sper = (a.nstiles + G - 1) / G;
        const uint32_t sfirst = min(a.nstiles, b * sper), slast = min(a.nstiles, sfirst + sper);
        uint32_t t = 0xFFFFFFFFu;
        TensorDesc d;
        for (uint32_t st = sfirst; st < slast; ++st) {
            if (t == 0xFFFFFFFFu || st >= d.stile0 + d.nstiles) {
                if (t != 0xFFFFFFFFu) flush_hist(sm, a.shist + (size_t)t * kHistBins, 1 << level_bits(0));
                __syncthreads();
                t = a.ntab ? owner(tab_stile0, st) : find_tensor<SampleSpace>(a.desc, a.T, st);
                d = a.desc[t];
            }
            if (d.kind == kKindSmall) continue;           // sampled by the CTA that finishes it
            const uint32_t ngroups = (d.n + 3u) >> 2;
            const uint32_t nsg = (ngroups + d.sstride - 1) / d.sstride;
            const uint64_t sg = (uint64_t)(st - d.stile0) * kBlock + tid;
            const uint64_t gi = sg * d.sstride;
            uint32_t key[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};     // = not a sample
            if (sg < nsg && gi < ngroups) {
                const uint32_t i0 = (uint32_t)gi * 4u;
                float gv[4], rv[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const bool v = i0 + e < d.n;
                    const uint32_t f = d.off + (v ? i0 + e : 0u);
                    gv[e] = v ? __ldg(a.g + f) : 0.f;
                    rv[e] = v ? ld_cg(a.r + f) : 0.f;
                }
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (i0 + e < d.n) key[e] = key_of(__fadd_rn(gv[e], rv[e]));
            }
#pragma unroll
            for (int e = 0; e < 4; ++e)          // (all lanes: the coarse counts are aggregated over the warp)
                hist_add_warp(sm.hist, key[e] == 0xFFFFFFFFu ? 0xFFFFFFFFu : key[e] >> level_shift(0), lane);
            a.skeys[(size_t)st * kBlock + tid] = make_uint4(key[0], key[1], key[2], key[3]);
        }
        if (t != 0xFFFFFFFFu) flush_hist(sm, a.shist + (size_t)t * kHistBins, 1 << level_bits(0));
    }
    grid_arrive(hdr);
    for (uint32_t q = G - 1u - b; q < a.n_small; q += G) {
        const uint32_t t = a.small_ids[q];
        const TensorDesc d = a.desc[t];
        small_threshold_body(sm, d, t, a.T, a.g, a.r, a.out_idx, a.out_val, a.out_count, hdr);
    }
    __syncthreads();
    for (int i = tid; i < 2048; i += kBlock) sm.hist[i] = 0u;
    if (!grid_wait(hdr, passed, &sm.ok, G)) return;
    phase_stamp(hdr, n_stamp, b);

    // ---------------------------------------------------------------- exact tau, one CTA per tensor
    for (uint32_t q = b; q < a.n_reg; q += G) {
        const uint32_t t = a.reg_ids[q];
        const TensorDesc d = a.desc[t];
        uint32_t bin0 = 0, above0 = 0, tau = 0xFFFFFFFFu;
        bool ok = block_select<(1 << level_bits(0)), false>(sm, a.shist + (size_t)t * kHistBins, d.srank, bin0, above0);
        const uint4* sk = a.skeys + (size_t)d.stile0 * kBlock;
        const uint32_t nk = d.nstiles * kBlock;
        uint32_t prefix = bin0, krem = d.srank - above0;
        int have = level_bits(0);                          // key bits fixed so far
        while (ok && have < 31) {
            const int w = min(11, 31 - have), sh = 31 - have - w;       // this level: bits [sh, sh + w)
            constexpr int kKeyBatch = 8;                   // loads in flight per thread: one CTA walks a whole tensor's keys
            for (uint32_t q0 = tid; q0 < nk; q0 += kKeyBatch * kBlock) {
                uint4 kv[kKeyBatch];
#pragma unroll
                for (int u = 0; u < kKeyBatch; ++u)
                    kv[u] = q0 + u * kBlock < nk ? ld_cg(sk + q0 + u * kBlock)
                                                 : make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);
#pragma unroll
                for (int u = 0; u < kKeyBatch; ++u) {
                    const uint32_t kk[4] = {kv[u].x, kv[u].y, kv[u].z, kv[u].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if ((kk[e] >> (sh + w)) == prefix) atomicAdd(&sm.hist[(kk[e] >> sh) & ((1u << w) - 1u)], 1u);
                }
            }
            __syncthreads();
            uint32_t bin, above;
            ok = block_select<2048, true>(sm, sm.hist, krem, bin, above);
            for (int i2 = tid; i2 < 2048; i2 += kBlock) sm.hist[i2] = 0u;
            __syncthreads();
            prefix = (prefix << w) | bin;
            krem -= above;
            have += w;
        }
        if (ok) tau = prefix;
        if (tid == 0) a.tsel[t].T = tau;                  // ~0: nothing is a hit (cannot happen for a valid plan)
    }
    if (!grid_barrier(hdr, passed, &sm.ok, G)) return;
    phase_stamp(hdr, n_stamp, b);

    // ---------------------------------------------------------------- fold + hits, segment by segment
    uint32_t nseg = 0;
    {
        const uint32_t my_off = warp * kWarpChunk + lane * 4;
        bool block_overflow = false;
        uint32_t cur = 0xFFFFFFFFu, tau = 0xFFFFFFFFu;
        TensorDesc d;
        for (uint32_t tile = first; tile < last; ++tile) {
            const uint32_t i = tile - first;
            if (cur == 0xFFFFFFFFu || tile >= d.tile0 + d.ntiles) {
                cur = a.ntab ? owner(tab_tile0, tile) : find_tensor(a.desc, a.T, tile);
                d = a.desc[cur];
                if (d.kind != kKindSmall) {
                    tau = ld_cg(&a.tsel[cur].T);
                    if (tid == 0) {
                        uint32_t* s = seg + (size_t)nseg * kSegWords;
                        const TileGeom tg0 = tile_geom(d, tile - d.tile0);
                        s[SG_T] = cur; s[SG_TILE0] = i; s[SG_NTILE] = min(last, d.tile0 + d.ntiles) - tile;
                        s[SG_BASE0] = (d.off & ~3u) + (tile - d.tile0) * (uint32_t)kTile; s[SG_BEGIN] = tg0.lo;
                        s[SG_OUT] = d.out_off; s[SG_K] = d.out_off + d.cap;           // SG_K: end of the tensor's slots
                    }
                    ++nseg;
                }
            }
            if (d.kind == kKindSmall) continue;
            const TileGeom tg = tile_geom(d, tile - d.tile0);
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
    }
    const uint32_t used = s_used;
    for (uint32_t i = tid; i < ntl; i += kBlock) {
        uint32_t tot = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) tot += rec[i * kWarps + w] & 1023u;
        a.tile_cnt[first + i] = tot;
    }
    if (!grid_barrier(hdr, passed, &sm.ok, G)) return;
    phase_stamp(hdr, n_stamp, b);

    if (ld_cg(&hdr->overflow) == 0u) {
        // ------------------------------------------------------------ slots and emission
        for (uint32_t sidx = 0; sidx < nseg; ++sidx) {
            uint32_t* s = seg + (size_t)sidx * kSegWords;
            const uint32_t t = s[SG_T];
            const TensorDesc d = a.desc[t];
            const bool head = first + s[SG_TILE0] == d.tile0;          // this CTA owns the tensor's first tile
            const uint32_t nbefore = first + s[SG_TILE0] - d.tile0;
            // hits in the tensor's earlier tiles; the owner of the first tile also totals the tensor
            uint32_t part = 0, whole = 0;
            for (uint32_t q = tid; q < (head ? d.ntiles : nbefore); q += kBlock) {
                const uint32_t v = ld_cg(a.tile_cnt + d.tile0 + q);
                whole += v;
                if (q < nbefore) part += v;
            }
            part = __reduce_add_sync(0xFFFFFFFFu, part);
            whole = __reduce_add_sync(0xFFFFFFFFu, whole);
            if (tid == 0) { s_cnt = 0u; sm.gt_sum = 0u; }
            __syncthreads();
            if (lane == 0) { if (part) atomicAdd(&s_cnt, part); if (whole) atomicAdd(&sm.gt_sum, whole); }
            __syncthreads();
            if (tid == 0) {
                s[SG_OUT] = d.out_off + s_cnt;
                if (head) {
                    const uint32_t hits = sm.gt_sum;
                    if (a.out_count != nullptr) { a.out_count[t] = min(hits, d.cap); a.out_count[a.T + t] = hits; }
                    if (hits > d.cap) record_status(hdr, 1 /*GC_W_TRUNCATED*/, t);
                }
            }
            __syncthreads();
        }
        // rec2[c] = slot of the first hit of chunk c (one warp walks each segment)
        for (uint32_t sidx = warp; sidx < nseg; sidx += kWarps) {
            const uint32_t* s = seg + (size_t)sidx * kSegWords;
            uint32_t run = s[SG_OUT];
            const uint32_t c0 = s[SG_TILE0] * kWarps, nc = s[SG_NTILE] * kWarps;
            for (uint32_t q0 = 0; q0 < nc; q0 += 32) {
                const uint32_t q = q0 + lane;
                const uint32_t v = q < nc ? (rec[c0 + q] & 1023u) : 0u;
                const uint32_t inc = warp_incl_scan(v, lane);
                if (q < nc) rec2[c0 + q] = run + inc - v;
                run += __shfl_sync(0xFFFFFFFFu, inc, 31);
            }
        }
        __syncthreads();
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
                uint32_t sx = nseg - 1u;                                   // segment of the hit
                while (sx > 0u && seg[(size_t)sx * kSegWords + SG_BEGIN] > pr[u].x) --sx;
                const uint32_t* s = seg + (size_t)sx * kSegWords;
                const uint32_t rel = pr[u].x - s[SG_BASE0];
                const uint32_t c = (s[SG_TILE0] + (rel >> 12)) * kWarps + ((rel >> 9) & (kWarps - 1u));
                const uint32_t slot = rec2[c] + (i - (rec[c] >> 10));
                if (slot < s[SG_K]) {
                    __stcs(a.out_idx + slot, pr[u].x);
                    __stcs(a.out_val + slot, __uint_as_float(pr[u].y));
                } else {
                    a.r[pr[u].x] = __uint_as_float(pr[u].y);        // beyond the capacity: stays in the residual
                }
            }
        }
        __syncthreads();
        phase_stamp(hdr, n_stamp, b);
        exit_stamp(hdr);
        return;
    }

    // ---------------------------------------------------------------- hit list overflowed (rare)
    for (uint32_t c = tid; c < ntl * kWarps; c += kBlock) {
        const uint32_t rc = rec[c], off = rc >> 10, cnt = rc & 1023u;
        for (uint32_t j = 0; j < cnt; ++j) {
            const uint2 pr = pool[off + j];
            a.r[pr.x] = __uint_as_float(pr.y);
        }
    }
    if (!grid_barrier(hdr, passed, &sm.ok, G)) return;
    phase_stamp(hdr, n_stamp, b);
    threshold_emit_body<false, true>(a.desc, a.T, a.ntiles, nullptr, a.r, a.out_idx, a.out_val, a.out_count, a.ws,
                                     a.tsel, 0u, 0);
}

// (three CTAs per SM: 80 registers and no spills beat four at 64 registers, see k_topk_single)
static __global__ void __launch_bounds__(kBlock, 3)
k_threshold_multi(const __grid_constant__ ThrMultiArgs a) {
    __shared__ BlockSmem sm;
    __shared__ uint32_t s_used, s_cnt;
    extern __shared__ __align__(16) unsigned char s_dyn[];
    threshold_multi_body(a, gridDim.x, blockIdx.x, sm, s_used, s_cnt, s_dyn);
}

// Several workers' threshold compress calls in one cooperative launch, one group of CTAs per
// worker (see k_topk_workers).
struct ThrWorkersArgs {
    uint32_t W, G;                               // workers in this launch, CTAs per worker
    ThrMultiArgs per[kWorkersPerLaunch];
};
static_assert(sizeof(ThrWorkersArgs) <= 4000, "kernel parameters stay below 4 KB");

static __global__ void __launch_bounds__(kBlock, 3)
k_threshold_workers(const __grid_constant__ ThrWorkersArgs wa) {
    __shared__ BlockSmem sm;
    __shared__ uint32_t s_used, s_cnt;
    __shared__ ThrMultiArgs s_args;               // this CTA's worker
    extern __shared__ __align__(16) unsigned char s_dyn[];
    const uint32_t w = blockIdx.x % wa.W, b = blockIdx.x / wa.W;
    {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(&wa.per[w]);
        uint32_t* dst = reinterpret_cast<uint32_t*>(&s_args);
        for (uint32_t i = threadIdx.x; i < sizeof(ThrMultiArgs) / 4; i += kBlock) dst[i] = src[i];
    }
    __syncthreads();
    threshold_multi_body(s_args, wa.G, b, sm, s_used, s_cnt, s_dyn);
}

}  // namespace gc
