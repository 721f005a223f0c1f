// Exact top-k of MANY tensors (layer-wise plans) in one cooperative launch.
//
// The scheme of the one-tensor kernel, applied per tensor: sample -> bracket [tau, tau_hi) and a
// guess tau_z of the threshold -> fold + candidates + band histogram -> band bin of the k-th
// key -> short list ranked by every CTA that needs it -> index-ordered emission; four grid
// barriers.  What differs:
//   * CTA b owns a contiguous run of tiles, so it sees one to a few tensors ("segments") and
//     keeps one small record per segment in shared memory;
//   * all histograms and short lists exist once per tensor in global memory; a CTA only looks
//     at those of its own segments;
//   * the sample is a coarse histogram (top 11 key bits) per tensor plus the kept sampled keys;
//     after the first barrier ONE CTA per tensor computes the bracket (the kept keys give tau a
//     second radix level; tau_hi is a bin edge; tau_z is interpolated inside its bin -- it is
//     only a guess) and publishes it, so the fold pass of the many CTAs that share a tensor
//     only reads three words per segment;
//   * the slot of a segment's first entry = what the tensor's earlier tiles send: the sum of
//     their published counts + the sent short-list entries that lie before the segment;
//   * tensors that fit one tile ("small") are finished by one CTA each between the arrival at
//     and the wait on the first barrier, dealt to the CTAs from the top (those have no sample
//     tiles);
//   * a tensor whose bracket missed, or whose band bin holds more than kMultiMidCap candidates,
//     is flagged and redone by the exact multi-pass kernels at the end (the others are not);
//     if a CTA's candidate region overflows, everything is redone.
#pragma once
#include "gc_single.cuh"

namespace gc {

constexpr uint32_t kMultiMidCap = kMidFast;      // short list per tensor (entries stay in registers)
constexpr uint32_t kSegWords = 16;               // shared-memory words per segment record
constexpr uint32_t kRefineTiles = 32;            // samples of up to this many sample tiles are ranked a second time
constexpr uint32_t kWarpMid = 128;               // short lists up to this length are settled by one warp

struct MultiArgs {
    const TensorDesc* desc;
    uint32_t T, ntiles, nstiles;
    uint32_t per;                    // tiles per CTA (contiguous run), at most
    uint32_t full_ctas;              // CTAs 0 .. full_ctas - 1 take `per` tiles each, the others share the rest evenly
    uint32_t pool_cap;               // candidate slots per CTA
    uint32_t pool_smem_words;        // words of shared memory reserved for one bit per candidate slot
    uint32_t ntab;                   // T if the tile tables fit in shared memory, else 0
    const uint32_t* small_ids;       // the tensors that fit one tile, the tiny ones (one warp each) first
    uint32_t n_small, n_tiny;
    const uint32_t* reg_ids;         // the tensors that are not small (and not empty)
    uint32_t n_reg;
    TensorSel* brk;                  // [T] bracket of every such tensor: .prefix = tau, .krem = tau_z, .T = shift
    const void* g;                   // fp32 or bf16, see the kernel's template argument
    float* r;
    uint32_t* out_idx;
    float* out_val;
    uint32_t* out_count;
    uint2* cand;                     // [gridDim.x * pool_cap]
    uint2* mid;                      // [T][kMultiMidCap] candidates inside the band bin of the threshold
    uint32_t* mid_n;                 // [T] their number (zeroed)
    uint32_t* shist;                 // [T][kHistBins] coarse sample histogram (zeroed)
    uint32_t* bhist;                 // [T][kHistBins] band histogram (zeroed)
    uint32_t* tile_cnt;              // [ntiles] candidates above the band bin, per tile
    uint4* skeys;                    // [nstiles * kBlock] the sampled keys, one group of four per entry
    WsView ws, gws;
    CleanArgs cl;                    // the control block is left clean for the next launch (early section: shist)
};

// segment record (one per tensor a CTA's tile run touches), kSegWords words in shared memory
enum : uint32_t {
    SG_T = 0, SG_TILE0, SG_NTILE, SG_BASE0, SG_BEGIN, SG_TAU, SG_TAUZ, SG_SHIFT,
    SG_A, SG_ABOVE, SG_M, SG_TKEY, SG_CUT, SG_OK, SG_OUT, SG_K
};

__device__ __forceinline__ void grid_arrive(WsHeader* hdr) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(&hdr->barrier, 1u);
    }
}
// second half of a barrier whose arrival was signalled with grid_arrive
__device__ __forceinline__ bool grid_wait(WsHeader* hdr, uint32_t& passed, int* s_ok, uint32_t G) {
    if (threadIdx.x == 0) {
        int ok = 1;
        const uint32_t target = (passed + 1u) * G;
        uint32_t spins = 0;
        while (ld_cg(&hdr->barrier) < target) {
            if (++spins > kSpinLimit || ((spins & 15u) == 0u && ld_cg(&hdr->abort) != 0u)) { ok = 0; break; }
            if (spins > 32) __nanosleep(spins > 4096 ? 400 : 60);
        }
        if (!ok) {
            record_status(hdr, -5 /*GC_E_TIMEOUT*/, 0xB0000000ull + passed);
            atomicExch(&hdr->abort, 1u);
        }
        __threadfence();
        *s_ok = ok;
    }
    __syncthreads();
    ++passed;
    return *s_ok != 0;
}
__device__ __forceinline__ bool grid_wait(WsHeader* hdr, uint32_t& passed, int* s_ok) {
    return grid_wait(hdr, passed, s_ok, gridDim.x);
}

// The whole compress of one worker by the G CTAs of one group (this CTA is number b of them);
// the group's barriers count on the worker's own workspace header.
template <typename GL>
__device__ __forceinline__ void topk_multi_body(const MultiArgs& a, const uint32_t G, const uint32_t b, BlockSmem& sm,
                                                uint32_t& s_used, uint32_t& s_cnt, unsigned char* s_dyn) {
    uint32_t* const rec = reinterpret_cast<uint32_t*>(s_dyn);                  // [per*kWarps] off<<10 | cnt
    uint32_t* const rec2 = rec + (size_t)a.per * kWarps;                       // [per*kWarps] counts, later slots
    uint32_t* const seg = rec2 + (size_t)a.per * kWarps;                       // [per][kSegWords]
    uint32_t* const sent_bits = seg + (size_t)a.per * kSegWords;               // [ceil(pool_cap / 32)]
    uint32_t* const tab_tile0 = sent_bits + (a.pool_smem_words);               // [ntab] first tile of every tensor
    uint32_t* const tab_stile0 = tab_tile0 + a.ntab;                           // [ntab] first sample tile
    uint2* const pool = a.cand + (size_t)b * a.pool_cap;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    WsHeader* hdr = a.ws.hdr;
    uint32_t passed = 0, n_stamp = 0;
    if (!clean_begin(a.cl, hdr, G, b, tid)) return;
    // The CTAs launched last are the youngest on their SMs and advance the slowest (see RowMap in
    // the one-tensor kernel), so whatever the full runs leave over is spread evenly over them.
    uint32_t first, last;
    if (b < a.full_ctas) {
        first = min(a.ntiles, b * a.per); last = min(a.ntiles, first + a.per);
    } else {
        const uint32_t s0 = min(a.ntiles, a.full_ctas * a.per), rest = a.ntiles - s0, nb = G - a.full_ctas;
        first = s0 + (uint32_t)(((unsigned long long)(b - a.full_ctas) * rest) / nb);
        last = s0 + (uint32_t)(((unsigned long long)(b - a.full_ctas + 1u) * rest) / nb);
    }
    const uint32_t ntl = last - first;                                         // own tiles
    for (int i = tid; i < 2048; i += kBlock) sm.hist[i] = 0u;
    for (uint32_t i = tid; i < ntl * kWarps; i += kBlock) { rec[i] = 0u; rec2[i] = 0u; }
    if (tid == 0) { s_used = 0u; s_cnt = 0u; }
    // first tile / first sample tile of every tensor, so that "which tensor owns this tile" is a
    // binary search in shared memory instead of a chain of dependent global loads
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

    // ---------------------------------------------------------------- sample: coarse histogram per tensor
    if (a.nstiles) {
        const uint32_t sper = (a.nstiles + G - 1) / G;
        const uint32_t sfirst = min(a.nstiles, b * sper), slast = min(a.nstiles, sfirst + sper);
        uint32_t t = 0xFFFFFFFFu;
        TensorDesc d;
        for (uint32_t st = sfirst; st < slast;) {
            if (t == 0xFFFFFFFFu || st >= d.stile0 + d.nstiles) {
                if (t != 0xFFFFFFFFu) flush_hist(sm, a.shist + (size_t)t * kHistBins, 1 << level_bits(0));
                __syncthreads();
                t = a.ntab ? owner(tab_stile0, st) : find_tensor<SampleSpace>(a.desc, a.T, st);
                d = a.desc[t];
            }
            // up to kSampleBatch sample tiles of this tensor at once: all their loads are in flight
            // together, so a CTA that owns several sample tiles (a group of CTAs that serves one of
            // several workers) pays one round trip for the batch instead of one per tile
            constexpr uint32_t kSampleBatch = 4;
            const uint32_t nb = min(kSampleBatch, min(slast, d.stile0 + d.nstiles) - st);
            const uint32_t ngroups = (d.n + 3u) >> 2;
            const uint32_t nsg = (ngroups + d.sstride - 1) / d.sstride;
            const bool vec_ok = (d.off & 3u) == 0u;           // the tensor's groups are 16-byte aligned in the flat buffers
            float gv[kSampleBatch][4], rv[kSampleBatch][4];
            uint32_t i0[kSampleBatch];
            bool live[kSampleBatch];
#pragma unroll
            for (uint32_t u = 0; u < kSampleBatch; ++u) {
                const uint64_t sg = (uint64_t)(st + u - d.stile0) * kBlock + tid;
                const uint64_t gi = sample_group(sg, d.sstride);
                live[u] = u < nb && sg < nsg && gi < ngroups;
                i0[u] = live[u] ? (uint32_t)gi * 4u : 0u;
                if (vec_ok && live[u] && i0[u] + 3u < d.n) {
                    // the whole group in one 16-byte load each (a quarter of the load instructions and
                    // of the sectors the L1 has to look up: the groups lie `sstride` x 16 bytes apart)
                    const float4 g4 = GL::ld4(a.g, d.off + i0[u]);
                    const float4 r4 = ld_cg(reinterpret_cast<const float4*>(a.r + d.off + i0[u]));
                    gv[u][0] = g4.x; gv[u][1] = g4.y; gv[u][2] = g4.z; gv[u][3] = g4.w;
                    rv[u][0] = r4.x; rv[u][1] = r4.y; rv[u][2] = r4.z; rv[u][3] = r4.w;
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const bool v = live[u] && i0[u] + e < d.n;
                        const uint32_t f = d.off + (v ? i0[u] + e : 0u);
                        gv[u][e] = v ? GL::ld1(a.g, f) : 0.f;
                        rv[u][e] = v ? ld_cg(a.r + f) : 0.f;
                    }
                }
            }
#pragma unroll
            for (uint32_t u = 0; u < kSampleBatch; ++u) {
                if (u < nb) {                             // (uniform over the CTA)
                    uint32_t key[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};     // = not a sample
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (live[u] && i0[u] + e < d.n) key[e] = key_of(__fadd_rn(gv[u][e], rv[u][e]));
                        hist_add_warp(sm.hist, key[e] == 0xFFFFFFFFu ? 0xFFFFFFFFu : key[e] >> level_shift(0), lane);
                    }
                    // the keys are kept: the fold pass ranks them a second time, and by then the residual
                    // they were computed from has been overwritten
                    if (d.nstiles <= kRefineTiles)
                        a.skeys[(size_t)(st + u) * kBlock + tid] = make_uint4(key[0], key[1], key[2], key[3]);
                }
            }
            st += nb;
        }
        if (t != 0xFFFFFFFFu) flush_hist(sm, a.shist + (size_t)t * kHistBins, 1 << level_bits(0));
    }
    grid_arrive(hdr);
    // small tensors need nothing from anyone: they fill the wait (CTAs from the top take them)
    for (uint32_t q8 = G - 1u - b; q8 * kWarps < a.n_tiny; q8 += G) {        // tiny ones: a warp each, eight at a time
        const uint32_t q = q8 * kWarps + (uint32_t)warp;
        if (q < a.n_tiny) {
            const uint32_t t = a.small_ids[q];
            const TensorDesc d = a.desc[t];
            tiny_tensor_warp<GL>(d.off, d.n, d.k, d.out_off, t, a.T, a.g, a.r, a.out_idx, a.out_val, a.out_count, lane);
        }
    }
    // (the other small ones start with the CTAs next to those that took the tiny ones)
    for (uint32_t q = a.n_tiny + (2u * G - 1u - b - ((a.n_tiny + kWarps - 1u) / kWarps) % G) % G; q < a.n_small; q += G) {
        const uint32_t t = a.small_ids[q];
        const TensorDesc d = a.desc[t];
        if (d.k <= kFewK) small_tensor_fewk<GL>(sm, d, t, a.T, a.g, a.r, a.out_idx, a.out_val, a.out_count);
        else small_tensor_body<GL>(sm, d, t, a.T, a.g, a.r, a.out_idx, a.out_val, a.out_count);
    }
    __syncthreads();
    for (int i = tid; i < 2048; i += kBlock) sm.hist[i] = 0u;
    if (!grid_wait(hdr, passed, &sm.ok, G)) return;
    phase_stamp(hdr, n_stamp, b);
    clean_in_use(hdr, b, tid);

    // ---------------------------------------------------------------- bracket per tensor, one CTA each
    // tau = the srank-th largest sampled key (22 bits when the kept keys allow the second radix
    // level, else the lower edge of its coarse bin), tau_hi = upper edge of the bin of the key
    // that stays below the expected rank by the same margin, tau_z inside the bin of the
    // expected rank itself; published as (tau, tau_z, shift of the band histogram).
    for (uint32_t q = b; q < a.n_reg; q += G) {
        const uint32_t cur = a.reg_ids[q];
        const TensorDesc d = a.desc[cur];
        uint32_t tau = 0, tau_z = 0;
        int shift = 0;
        {
            uint32_t tau_hi = 0x80000000u;
            if (d.sstride != 0u) {
                const uint32_t ngroups = (d.n + 3u) >> 2;
                const float msamp = 4.0f * (float)((ngroups + d.sstride - 1) / d.sstride);
                const float ks = (float)d.k * msamp / (float)d.n;
                const float hi = floorf(ks - 6.0f * sqrtf(ks) - 8.0f);
                // (a sample too small for that margin: the largest sampled key bounds the band instead)
                const uint32_t want[3] = {d.srank, hi >= 1.0f ? (uint32_t)hi : 1u, max(1u, (uint32_t)ceilf(ks))};
                Picked pk[3];
                block_select_multi<(1 << level_bits(0)), 3>(sm, a.shist + (size_t)cur * kHistBins, want, pk);
                if (pk[0].ok) tau = pk[0].bin << level_shift(0);
                if (pk[0].ok && d.nstiles <= kRefineTiles) {
                    // second radix level of the lower bracket over the kept sample keys:
                    // tau gets 22 significant bits
                    const uint4* sk = a.skeys + (size_t)d.stile0 * kBlock;
                    const uint32_t nk = d.nstiles * kBlock, bin0 = pk[0].bin;
                    for (uint32_t q0 = tid; q0 < nk; q0 += 4 * kBlock) {
                        uint4 kv[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            kv[u] = q0 + u * kBlock < nk ? ld_cg(sk + q0 + u * kBlock)
                                                         : make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const uint32_t kk[4] = {kv[u].x, kv[u].y, kv[u].z, kv[u].w};
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if ((kk[e] >> level_shift(0)) == bin0)
                                    atomicAdd(&sm.hist[(kk[e] >> (level_shift(0) - 11)) & 2047u], 1u);
                        }
                    }
                    __syncthreads();
                    uint32_t bin1, above1;
                    const bool ok1 = block_select<2048, true>(sm, sm.hist, d.srank - pk[0].above, bin1, above1);
                    for (int i2 = tid; i2 < 2048; i2 += kBlock) sm.hist[i2] = 0u;
                    __syncthreads();
                    if (ok1) tau |= bin1 << (level_shift(0) - 11);
                }
                if (pk[1].ok) tau_hi = (pk[1].bin + 1u) << level_shift(0);
                if (pk[2].ok) {
                    const float pos = ((float)(want[2] - pk[2].above) - 0.5f) / (float)pk[2].count;   // from the top of the bin
                    tau_z = (pk[2].bin << level_shift(0)) +
                            (uint32_t)((1.0f - pos) * (float)((1u << level_shift(0)) - 1u));
                }
            }
            if (tau_z < tau) tau_z = tau;
            if (tau_hi <= tau) tau_hi = 0x80000000u;
            shift = 0;
            while (((tau_hi - tau) >> shift) > 2046u) ++shift;
        }
        if (tid == 0) { a.brk[cur].prefix = tau; a.brk[cur].krem = tau_z; a.brk[cur].T = (uint32_t)shift; }
    }
    if (!grid_barrier(hdr, passed, &sm.ok, G)) return;
    phase_stamp(hdr, n_stamp, b);
    clean_early(a.cl, G, b, tid);      // the sample histograms have had their last reader (the brackets)

    // ---------------------------------------------------------------- fold + candidates, segment by segment
    uint32_t nseg = 0;
    {
        const uint32_t my_off = warp * kWarpChunk + lane * 4;
        bool block_overflow = false, open = false;
        uint32_t cur = 0xFFFFFFFFu, tau = 0, tau_z = 0;
        int shift = 0;
        TensorDesc d;
        for (uint32_t tile = first; tile < last; ++tile) {
            const uint32_t i = tile - first;
            if (cur == 0xFFFFFFFFu || tile >= d.tile0 + d.ntiles) {
                if (open) flush_hist(sm, a.bhist + (size_t)cur * kHistBins, 2048);
                open = false;
                cur = a.ntab ? owner(tab_tile0, tile) : find_tensor(a.desc, a.T, tile);
                d = a.desc[cur];
                if (d.kind != kKindSmall) {
                    // bracket of this tensor, published by the CTA that computed it
                    tau = ld_cg(&a.brk[cur].prefix);
                    tau_z = ld_cg(&a.brk[cur].krem);
                    shift = (int)ld_cg(&a.brk[cur].T);
                    if (tid == 0) {
                        uint32_t* s = seg + (size_t)nseg * kSegWords;
                        const TileGeom tg0 = tile_geom(d, tile - d.tile0);
                        s[SG_T] = cur; s[SG_TILE0] = i; s[SG_NTILE] = min(last, d.tile0 + d.ntiles) - tile;
                        s[SG_BASE0] = (d.off & ~3u) + (tile - d.tile0) * (uint32_t)kTile; s[SG_BEGIN] = tg0.lo;
                        s[SG_TAU] = tau; s[SG_TAUZ] = tau_z; s[SG_SHIFT] = (uint32_t)shift;
                        s[SG_OK] = 1u; s[SG_OUT] = d.out_off; s[SG_K] = d.k;
                    }
                    ++nseg;
                    open = true;
                }
            }
            if (d.kind == kKindSmall) continue;          // finished by its own CTA
            const TileGeom tg = tile_geom(d, tile - d.tile0);
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
                    if (!interior) hm |= (uint32_t)(key >= tau_z) << (4 * j + e);
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
            const uint32_t em = fits ? cm : 0u;             // goes to the candidate list
            const uint32_t zm = fits ? (hm & cm) : 0u;      // ... and leaves +0 in the residual (probably sent)
            if (interior) {
                // +0 where the key reaches tau_z (implies a candidate: tau_z >= tau), a elsewhere; a chunk
                // that did not fit keeps all its values (no key reaches 2^31)
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
            const bool staged = wtot <= (uint32_t)kEmitStage;
            if (fits && wtot != 0u) {
                // one round per candidate of the lane that has the most, instead of sixteen predicated
                // blocks that every warp walks through (see the one-tensor kernel)
                for (uint32_t m = em; m != 0u; m &= m - 1u) {
                    const uint32_t bq = (uint32_t)__ffs((int)m) - 1u, j = bq >> 2;      // element 4 j + e of this thread
                    float s8[8], s4[4];                                                 // its value by a select tree
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
        if (open) flush_hist(sm, a.bhist + (size_t)cur * kHistBins, 2048);
        if (__syncthreads_or(block_overflow ? 1 : 0)) {
            if (tid == 0) atomicExch(&hdr->overflow, 1u);
        }
        if (tid == 0) atomicAdd(&hdr->cand_total, min(s_used, a.pool_cap));
    }
    const uint32_t used = s_used;      // read linearly only when no chunk anywhere overflowed
    if (!grid_barrier(hdr, passed, &sm.ok, G)) return;
    phase_stamp(hdr, n_stamp, b);

    // segment of a candidate: the last one that begins at or before its index
    auto seg_of = [&](uint32_t idx) -> uint32_t* {
        uint32_t s = nseg - 1u;
        while (s > 0u && seg[(size_t)s * kSegWords + SG_BEGIN] > idx) --s;
        return seg + (size_t)s * kSegWords;
    };
    auto chunk_of = [&](const uint32_t* s, uint32_t idx) -> uint32_t {
        const uint32_t rel = idx - s[SG_BASE0];
        return (s[SG_TILE0] + (rel >> 12)) * kWarps + ((rel >> 9) & (kWarps - 1u));
    };

    const bool overflowed = ld_cg(&hdr->overflow) != 0u;
    if (!overflowed && nseg != 0u) {
        // ------------------------------------------------------------ band bin per segment, counts above it
        for (uint32_t sidx = (uint32_t)warp; sidx < nseg; sidx += kWarps) {      // a warp per segment, all at once
            uint32_t* s = seg + (size_t)sidx * kSegWords;
            const uint32_t t = s[SG_T];
            const Picked pa = warp_select_2048(a.bhist + (size_t)t * kHistBins, s[SG_K], lane);
            const bool ok = pa.ok && pa.count <= kMultiMidCap;
            if (lane == 0) {
                s[SG_A] = pa.bin; s[SG_ABOVE] = pa.above; s[SG_M] = pa.count; s[SG_OK] = ok ? 1u : 0u;
                if (!ok) {          // every CTA that sees this tensor decides the same; count it once
                    const uint32_t old = atomicOr(&a.ws.sel[t].flags, kSelFailed);
                    if ((old & kSelFailed) == 0u) atomicAdd(&hdr->n_failed, 1u);
                }
            }
        }
        __syncthreads();
        auto classify = [&](const uint2& pr) {
            const uint32_t* s = seg_of(pr.x);
            if (s[SG_OK] == 0u) return;
            const uint32_t bin = min(((pr.y & kKeyMask) - s[SG_TAU]) >> s[SG_SHIFT], 2047u);
            if (bin > s[SG_A]) {
                atomicAdd(&rec2[chunk_of(s, pr.x)], 1u);
            } else if (bin == s[SG_A]) {
                const uint32_t slot = atomicAdd(a.mid_n + s[SG_T], 1u);
                if (slot < kMultiMidCap) a.mid[(size_t)s[SG_T] * kMultiMidCap + slot] = pr;
            }
        };
        for (uint32_t i0 = tid; i0 < used; i0 += 4 * kBlock) {      // four loads in flight per thread
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
        for (uint32_t i = tid; i < ntl; i += kBlock) {
            uint32_t tot = 0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) tot += rec2[i * kWarps + w];
            a.tile_cnt[first + i] = tot;
        }
    }
    if (!grid_barrier(hdr, passed, &sm.ok, G)) return;
    phase_stamp(hdr, n_stamp, b);

    if (!overflowed) {
        if (nseg != 0u) {
            // -------------------------------------------------------- threshold, tie cut and slots per segment
            // Short lists of up to kWarpMid entries (nearly all: a band bin holds a handful of
            // candidates) are settled by a warp each, all segments of the CTA at once and without a
            // block-wide barrier: every entry's place in the order (key descending, index ascending)
            // is counted directly against all others, which settles threshold and tie cut in one go.
            for (uint32_t sidx = (uint32_t)warp; sidx < nseg; sidx += kWarps) {
                uint32_t* s = seg + (size_t)sidx * kSegWords;
                const uint32_t m = s[SG_M];
                if (s[SG_OK] == 0u || m > kWarpMid) continue;
                const uint32_t t = s[SG_T];
                const TensorDesc d = a.desc[t];
                const uint2* mid = a.mid + (size_t)t * kMultiMidCap;
                uint2 e[kWarpMid / 32];
#pragma unroll
                for (uint32_t u = 0; u < kWarpMid / 32; ++u)
                    e[u] = u * 32u + lane < m ? ld_cg(mid + u * 32u + lane) : make_uint2(0xFFFFFFFFu, 0u);
                // candidates above the band bin in the tensor's tiles before this segment
                const uint32_t nbefore = first + s[SG_TILE0] - d.tile0;
                uint32_t part = 0;
                for (uint32_t q = lane; q < nbefore; q += 32u) part += ld_cg(a.tile_cnt + d.tile0 + q);
                part = __reduce_add_sync(0xFFFFFFFFu, part);
                const uint32_t krem = s[SG_K] - s[SG_ABOVE];             // entries of the short list that are sent (1 .. m)
                // place of every own entry: entries that come before it in the order
                uint32_t place[kWarpMid / 32];
#pragma unroll
                for (uint32_t u = 0; u < kWarpMid / 32; ++u) place[u] = 0u;
#pragma unroll
                for (uint32_t uo = 0; uo < kWarpMid / 32; ++uo) {
                    if (uo * 32u >= m) break;                            // (uniform)
                    const uint32_t lim = min(32u, m - uo * 32u);
                    for (uint32_t l = 0; l < lim; ++l) {
                        const uint32_t ox = __shfl_sync(0xFFFFFFFFu, e[uo].x, (int)l);
                        const uint32_t ok = __shfl_sync(0xFFFFFFFFu, e[uo].y, (int)l) & kKeyMask;
#pragma unroll
                        for (uint32_t u = 0; u < kWarpMid / 32; ++u) {
                            const uint32_t key = e[u].y & kKeyMask;
                            place[u] += (ok > key || (ok == key && ox < e[u].x)) ? 1u : 0u;
                        }
                    }
                }
                // the last entry that is sent gives the threshold key and the tie cut; sent entries before
                // the segment shift its first slot, inside it they join the count of their chunk
                const uint32_t seg_end = s[SG_BASE0] + s[SG_NTILE] * (uint32_t)kTile;
                uint32_t before = 0, tk = 0, cut = 0;
                bool have = false;
#pragma unroll
                for (uint32_t u = 0; u < kWarpMid / 32; ++u) {
                    if (u * 32u + lane >= m) continue;
                    if (place[u] == krem - 1u) { have = true; tk = e[u].y & kKeyMask; cut = e[u].x; }
                    if (place[u] < krem) {
                        if (e[u].x < s[SG_BEGIN]) ++before;
                        else if (e[u].x < seg_end) atomicAdd(&rec2[chunk_of(s, e[u].x)], 1u);
                    }
                }
                before = __reduce_add_sync(0xFFFFFFFFu, before);
                const unsigned who = __ballot_sync(0xFFFFFFFFu, have);
                const bool good = who != 0u;                             // (the list holds at least krem entries)
                const int src = good ? __ffs(who) - 1 : 0;
                tk = __shfl_sync(0xFFFFFFFFu, tk, src); cut = __shfl_sync(0xFFFFFFFFu, cut, src);
                __syncwarp();
                if (lane == 0) {
                    s[SG_TKEY] = tk; s[SG_CUT] = cut;
                    s[SG_OUT] = d.out_off + part + before;             // slot of the segment's first sent entry
                    if (!good) {        // cannot happen unless the list changed under us: report, send nothing
                        s[SG_OK] = 0u;
                        record_status(hdr, -1 /*GC_E_INVALID*/, 0xE0000000ull + t);
                    } else if (a.out_count != nullptr && first + s[SG_TILE0] == d.tile0) {
                        a.out_count[t] = d.k; a.out_count[a.T + t] = d.k;
                    }
                }
            }
            __syncthreads();
            // longer short lists: the whole CTA, one segment after the other (radix select in shared memory)
            for (uint32_t sidx = 0; sidx < nseg; ++sidx) {
                uint32_t* s = seg + (size_t)sidx * kSegWords;
                if (s[SG_OK] == 0u || s[SG_M] <= kWarpMid) continue;
                const uint32_t t = s[SG_T], m = s[SG_M];
                const TensorDesc d = a.desc[t];
                const uint2* mid = a.mid + (size_t)t * kMultiMidCap;
                uint2 e[kMidRegs];
#pragma unroll
                for (uint32_t u = 0; u < kMidRegs; ++u)
                    e[u] = u * kBlock + tid < m ? ld_cg(mid + u * kBlock + tid) : make_uint2(0u, 0u);
                // candidates above the band bin in the tensor's tiles before this segment
                const uint32_t nbefore = first + s[SG_TILE0] - d.tile0;
                uint32_t part = 0;
                for (uint32_t q = tid; q < nbefore; q += kBlock) part += ld_cg(a.tile_cnt + d.tile0 + q);
                part = __reduce_add_sync(0xFFFFFFFFu, part);
                if (tid == 0) s_cnt = 0u;
                __syncthreads();
                if (lane == 0 && part) atomicAdd(&s_cnt, part);
                const uint32_t shift = s[SG_SHIFT], A = s[SG_A];
                const uint32_t binlo = s[SG_TAU] + (A << shift);
                uint32_t v_sel, mid_gt, n_eq, idx_cut = 0xFFFFFFFFu;
                const uint32_t krem = s[SG_K] - s[SG_ABOVE];
                bool good = short_list_select(sm, e, mid, m, A == 2047u ? 31 : max((int)shift, 1), krem,
                                              [&](const uint2& pr, uint32_t& v) { v = (pr.y & kKeyMask) - binlo; return true; },
                                              v_sel, mid_gt, n_eq);
                const uint32_t Tkey = binlo + v_sel;
                const uint32_t m_eq = krem - mid_gt;
                if (good && n_eq > m_eq) {
                    uint32_t v_idx, x0, x1;
                    good = short_list_select(sm, e, mid, m, 32, m_eq,
                                             [&](const uint2& pr, uint32_t& v) { v = ~pr.x; return (pr.y & kKeyMask) == Tkey; },
                                             v_idx, x0, x1);
                    idx_cut = ~v_idx;
                }
                // sent short-list entries: before the segment they shift its first slot, inside it
                // they join the count of their chunk
                const uint32_t seg_end = s[SG_BASE0] + s[SG_NTILE] * (uint32_t)kTile;
#pragma unroll
                for (uint32_t u = 0; u < kMidRegs; ++u) {
                    if (!(good && u * kBlock + tid < m)) continue;
                    const uint32_t key = e[u].y & kKeyMask;
                    if (!(key > Tkey || (key == Tkey && e[u].x <= idx_cut))) continue;
                    if (e[u].x < s[SG_BEGIN]) atomicAdd(&s_cnt, 1u);
                    else if (e[u].x < seg_end) atomicAdd(&rec2[chunk_of(s, e[u].x)], 1u);
                }
                __syncthreads();
                if (tid == 0) {
                    s[SG_TKEY] = Tkey; s[SG_CUT] = idx_cut;
                    s[SG_OUT] = d.out_off + s_cnt;                     // slot of the segment's first sent entry
                    if (!good) {        // cannot happen unless the list changed under us: report, send nothing
                        s[SG_OK] = 0u;
                        record_status(hdr, -1 /*GC_E_INVALID*/, 0xE0000000ull + t);
                    } else if (a.out_count != nullptr && first + s[SG_TILE0] == d.tile0) {
                        a.out_count[t] = d.k; a.out_count[a.T + t] = d.k;
                    }
                }
                __syncthreads();
            }
            // rec2[c] = output slot of the first sent candidate of chunk c (one warp walks each segment)
            for (uint32_t sidx = warp; sidx < nseg; sidx += kWarps) {
                const uint32_t* s = seg + (size_t)sidx * kSegWords;
                if (s[SG_OK] == 0u) continue;
                uint32_t run = s[SG_OUT];
                const uint32_t c0 = s[SG_TILE0] * kWarps, nc = s[SG_NTILE] * kWarps;
                for (uint32_t q0 = 0; q0 < nc; q0 += 32) {
                    const uint32_t q = q0 + lane;
                    const uint32_t v = q < nc ? rec2[c0 + q] : 0u;
                    const uint32_t inc = warp_incl_scan(v, lane);
                    if (q < nc) rec2[c0 + q] = run + inc - v;
                    run += __shfl_sync(0xFFFFFFFFu, inc, 31);
                }
            }
            __syncthreads();
        }
        phase_stamp(hdr, n_stamp, b);
        // sent flags of the CTA's candidates in list order, one bit each
        auto sent_of = [&](const uint32_t* s, const uint2& pr) {
            const uint32_t key = pr.y & kKeyMask;
            return s[SG_OK] != 0u && (key > s[SG_TKEY] || (key == s[SG_TKEY] && pr.x <= s[SG_CUT]));
        };
        const uint32_t nwords = (used + 31u) >> 5;
        for (uint32_t i0 = 0; i0 < nwords * 32u; i0 += kBlock) {
            const uint32_t i = i0 + tid;
            if (i0 + (tid & ~31) >= nwords * 32u) continue;          // whole warp past the end
            bool sent = false;
            if (i < used) {
                const uint2 pr = pool[i];
                sent = sent_of(seg_of(pr.x), pr);
            }
            const unsigned sb = __ballot_sync(0xFFFFFFFFu, sent);
            if (lane == 0) sent_bits[i >> 5] = sb;
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
                const uint32_t* s = seg_of(pr[u].x);
                // the fold pass left +0 in the residual iff the key reached tau_z
                const bool zeroed = (pr[u].y & kKeyMask) >= s[SG_TAUZ];
                if (!sent_of(s, pr[u])) {          // also every candidate of a tensor that is redone
                    if (zeroed) a.r[pr[u].x] = __uint_as_float(pr[u].y);     // value goes back
                    continue;
                }
                if (!zeroed) a.r[pr[u].x] = 0.0f;
                const uint32_t c = chunk_of(s, pr[u].x);
                const uint32_t p0 = rec[c] >> 10;                  // first list position of the chunk
                uint32_t before;
                if ((p0 >> 5) == (i >> 5)) {
                    before = __popc((sent_bits[i >> 5] & ((1u << (i & 31u)) - 1u)) >> (p0 & 31u));
                } else {
                    before = __popc(sent_bits[p0 >> 5] >> (p0 & 31u)) + __popc(sent_bits[i >> 5] & ((1u << (i & 31u)) - 1u));
                    for (uint32_t w = (p0 >> 5) + 1u; w < (i >> 5); ++w) before += __popc(sent_bits[w]);
                }
                const uint32_t slot = rec2[c] + before;
                a.out_idx[slot] = pr[u].x;
                a.out_val[slot] = __uint_as_float(pr[u].y);
            }
        }
        __syncthreads();
        phase_stamp(hdr, n_stamp, b);
        exit_stamp(hdr);
        if (ld_cg(&hdr->n_failed) == 0u) { leave_clean(a.cl, hdr, G, tid); return; }
    } else {
        // a candidate region overflowed: every recorded candidate gets its value back
        for (uint32_t c = tid; c < ntl * kWarps; c += kBlock) {
            const uint32_t rc = rec[c], off = rc >> 10, cnt = rc & 1023u;
            for (uint32_t j = 0; j < cnt; ++j) {
                const uint2 pr = pool[off + j];
                a.r[pr.x] = __uint_as_float(pr.y);
            }
        }
    }

    // ---------------------------------------------------------------- exact redo (rare)
    // of the flagged tensors, or of all of them after an overflow: r holds a = g + r for them again
    if (!grid_barrier(hdr, passed, &sm.ok, G)) return;
    phase_stamp(hdr, n_stamp, b);
    hist_body<0, SRC_RESID>(sm, a.desc, a.T, a.ntiles, nullptr, a.r, a.gws, G, b);
    if (!grid_barrier(hdr, passed, &sm.ok, G)) return;
    hist_body<1, SRC_RESID>(sm, a.desc, a.T, a.ntiles, nullptr, a.r, a.gws, G, b);
    if (!grid_barrier(hdr, passed, &sm.ok, G)) return;
    hist_body<2, SRC_RESID>(sm, a.desc, a.T, a.ntiles, nullptr, a.r, a.gws, G, b);
    if (!grid_barrier(hdr, passed, &sm.ok, G)) return;
    compact_body(sm, a.desc, a.T, a.ntiles, a.r, a.out_idx, a.out_val, a.out_count, a.gws, 0);
    __syncthreads();
    leave_clean(a.cl, hdr, G, tid);
}

template <typename GL>
// (three CTAs per SM: 80 registers and no spills beat four at 64 registers, see k_topk_single)
static __global__ void __launch_bounds__(kBlock, 3)
k_topk_multi(const __grid_constant__ MultiArgs a) {
    __shared__ BlockSmem sm;
    __shared__ uint32_t s_used, s_cnt;
    extern __shared__ __align__(16) unsigned char s_dyn[];
    topk_multi_body<GL>(a, gridDim.x, blockIdx.x, sm, s_used, s_cnt, s_dyn);
}

// Several workers' compress calls in ONE cooperative launch: the grid is cut into one group of
// CTAs per worker (CTA x serves worker x mod W as number x / W of its group, so every worker's
// CTAs are spread over all SMs), and each group runs the kernel above on its own gradient,
// residual, outputs and workspace.  Nothing is shared between the groups, not even a barrier:
// a group's phases wait only for that worker's CTAs, so while one worker's CTAs sit in a
// barrier the SMs stream another worker's tiles.
constexpr uint32_t kWorkersPerLaunch = 12;       // per-worker argument blocks travel as kernel parameters
struct WorkersArgs {
    uint32_t W, G;                               // workers in this launch, CTAs per worker
    MultiArgs per[kWorkersPerLaunch];
};
static_assert(sizeof(WorkersArgs) <= 4000, "kernel parameters stay below 4 KB");

template <typename GL>
static __global__ void __launch_bounds__(kBlock, 3)
k_topk_workers(const __grid_constant__ WorkersArgs wa) {
    __shared__ BlockSmem sm;
    __shared__ uint32_t s_used, s_cnt;
    __shared__ MultiArgs s_args;                  // this CTA's worker (dynamic indexing of the parameters happens once)
    extern __shared__ __align__(16) unsigned char s_dyn[];
    const uint32_t w = blockIdx.x % wa.W, b = blockIdx.x / wa.W;
    {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(&wa.per[w]);
        uint32_t* dst = reinterpret_cast<uint32_t*>(&s_args);
        for (uint32_t i = threadIdx.x; i < sizeof(MultiArgs) / 4; i += kBlock) dst[i] = src[i];
    }
    __syncthreads();
    topk_multi_body<GL>(s_args, wa.G, b, sm, s_used, s_cnt, s_dyn);
}

}  // namespace gc
