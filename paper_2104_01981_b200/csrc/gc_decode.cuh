// Tiled decode: dense_out = (zero | dense_out) + sum over workers of their sparse sets, with the
// additions applied in worker order 0..W-1 for every element (bit-reproducible).
//
// Every warp owns a contiguous run of 1024-element tiles of the dense buffer.  A tile is built
// in shared memory -- cleared or loaded, then the entries of each worker that fall inside it
// are added in worker order -- and leaves as one 4 KB bulk asynchronous copy (shared -> global),
// so the dense buffer is written exactly once, fully coalesced, and never read in zero-first
// mode.  Each worker's list is sorted by index, so a warp walks it with a cursor; the cursor's
// starting point is found once per warp by a cooperative multi-way search.
#pragma once
#include "gc_common.cuh"

namespace gc {

constexpr int kDecTile = 1024;               // floats per warp tile
constexpr int kDecBlock = 256;
constexpr int kDecWarps = kDecBlock / 32;
constexpr int kDecRounds = 4;                // entries a lane pre-loads per worker and tile

struct DecodeLists {
    const uint32_t* idx[64];
    const float* val[64];
};

__device__ __forceinline__ void bulk_store_tile(float* gdst, const float* ssrc, uint32_t bytes) {
    // generic-proxy writes to shared memory must be fenced before the async proxy reads them
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    const uint32_t sa = (uint32_t)__cvta_generic_to_shared(ssrc);
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(gdst), "r"(sa), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// First position p in idx[0..cnt) with idx[p] >= key, found by `L` cooperating lanes (L a power
// of two; the lanes of one search are consecutive and `sub` is the lane's rank among them).
__device__ __forceinline__ uint32_t group_lower_bound(const uint32_t* __restrict__ idx, uint32_t cnt,
                                                      uint32_t key, int L, int sub, unsigned gmask, bool live) {
    uint32_t lo = 0, hi = live ? cnt : 0u;               // answer in [lo, hi]
    // every lane of the warp runs the same number of rounds (worst case over the warp)
    while (__any_sync(0xFFFFFFFFu, hi > lo)) {
        const uint32_t span = hi - lo;
        // probe L points that split [lo, hi) into L + 1 parts
        const uint32_t p = lo + (uint32_t)(((unsigned long long)span * (uint32_t)(sub + 1)) / (uint32_t)(L + 1));
        const bool valid = hi > lo && p < hi;
        const uint32_t v = valid ? __ldg(idx + p) : 0xFFFFFFFFu;
        const bool ge = !valid || v >= key;              // monotone in sub: false..false true..true
        const unsigned b = __ballot_sync(0xFFFFFFFFu, ge) & gmask;
        const unsigned nb = __ballot_sync(0xFFFFFFFFu, !ge) & gmask;
        if (hi > lo) {
            // first probing lane that saw >= key bounds hi; last that saw < key bounds lo
            const int first_lane = __ffs(gmask) - 1;
            if (b) {
                const int fl = __ffs(b) - 1 - first_lane;                  // sub of first ">="
                const uint32_t pf = lo + (uint32_t)(((unsigned long long)span * (uint32_t)(fl + 1)) / (uint32_t)(L + 1));
                if (pf < hi) hi = pf;
            }
            if (nb) {
                const int ll = 31 - __clz(nb) - first_lane;               // sub of last "<"
                const uint32_t pl = lo + (uint32_t)(((unsigned long long)span * (uint32_t)(ll + 1)) / (uint32_t)(L + 1));
                if (pl + 1 > lo) lo = min(pl + 1, hi);
            }
            if (!b && !nb) hi = lo;
        }
    }
    return lo;
}

static __global__ void __launch_bounds__(kDecBlock)
k_decode_tiles(DecodeLists ls, uint32_t W, uint32_t cnt, uint32_t total_n, float* __restrict__ out,
               int zero_first, int use_bulk, WsHeader* hdr) {
    __shared__ __align__(128) float s_tile[kDecWarps][kDecTile];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float* tilebuf = s_tile[warp];
    const uint32_t ntl = (total_n + kDecTile - 1) / kDecTile;
    const uint32_t nwarps = gridDim.x * kDecWarps, gw = blockIdx.x * kDecWarps + warp;
    const uint32_t per = (ntl + nwarps - 1) / nwarps;
    const uint32_t t0 = gw * per, t1 = min(ntl, t0 + per);
    if (t0 >= t1) return;

    // lanes per worker in the fast path: E consecutive lanes serve one worker
    int Wp = 1;
    while (Wp < (int)min(W, 32u)) Wp <<= 1;
    const int E = 32 / Wp;
    const int sub = lane % E;
    // cursors: this lane keeps the cursor of worker (pass * Wp + lane / E) for each pass of Wp workers
    const int passes = (int)((W + Wp - 1) / Wp);                      // 1 or 2 (W <= 64)
    uint32_t cur[2] = {0u, 0u};
    const unsigned gmask = (E == 32) ? 0xFFFFFFFFu : (((1u << E) - 1u) << (lane - sub));
    const uint32_t key0 = t0 * (uint32_t)kDecTile;
    for (int ps = 0; ps < passes; ++ps) {
        const uint32_t w = (uint32_t)(ps * Wp + lane / E);
        const bool live = w < W;
        cur[ps] = group_lower_bound(live ? ls.idx[w] : ls.idx[0], cnt, key0, E, sub, gmask, live);
    }

    for (uint32_t tl = t0; tl < t1; ++tl) {
        const uint32_t lo = tl * (uint32_t)kDecTile;
        const uint32_t hi = min(total_n, lo + (uint32_t)kDecTile);
        const bool full = hi - lo == (uint32_t)kDecTile;
        // stage the tile
        if (zero_first) {
#pragma unroll
            for (int q = 0; q < kDecTile / 128; ++q)
                *reinterpret_cast<float4*>(tilebuf + q * 128 + lane * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
        } else if (full && use_bulk) {
#pragma unroll
            for (int q = 0; q < kDecTile / 128; ++q)
                *reinterpret_cast<float4*>(tilebuf + q * 128 + lane * 4) =
                    *reinterpret_cast<const float4*>(out + lo + q * 128 + lane * 4);
        } else {
            for (uint32_t q = lane; q < (uint32_t)kDecTile; q += 32) tilebuf[q] = (lo + q < hi) ? out[lo + q] : 0.f;
        }
        __syncwarp();
        for (int ps = 0; ps < passes; ++ps) {
            const uint32_t w = (uint32_t)(ps * Wp + lane / E);
            const bool live = w < W;
            // fast path: the first kDecRounds * E entries at the cursor of every worker, loaded together
            uint32_t ix[kDecRounds];
            float v[kDecRounds];
            uint32_t nin = 0;
#pragma unroll
            for (int rd = 0; rd < kDecRounds; ++rd) {
                const uint32_t p = cur[ps] + (uint32_t)(rd * E + sub);
                ix[rd] = 0xFFFFFFFFu; v[rd] = 0.f;
                if (live && p < cnt) { ix[rd] = __ldg(ls.idx[w] + p); v[rd] = __ldg(ls.val[w] + p); }
            }
#pragma unroll
            for (int rd = 0; rd < kDecRounds; ++rd) nin += ix[rd] < hi;   // sorted lists: the ins are a prefix
            // a worker whose loaded entries all fall inside may have more: then this tile takes
            // the strictly sequential path below so that worker order is kept for every element
            const bool maybe_more = (ix[kDecRounds - 1] < hi) && sub == E - 1;
            if (!__any_sync(0xFFFFFFFFu, maybe_more)) {
                for (int q = 0; q < Wp; ++q) {            // apply in worker order
                    if (lane / E == q) {
#pragma unroll
                        for (int rd = 0; rd < kDecRounds; ++rd) {
                            if (ix[rd] < hi) {
                                if (ix[rd] >= lo) tilebuf[ix[rd] - lo] = __fadd_rn(tilebuf[ix[rd] - lo], v[rd]);
                                else record_status(hdr, -1 /*GC_E_INVALID*/, cur[ps]);      // unsorted input
                            }
                        }
                    }
                    __syncwarp();
                }
                uint32_t tot = nin;                       // sum over the E lanes of the group
                for (int o = 1; o < E; o <<= 1) tot += __shfl_xor_sync(0xFFFFFFFFu, tot, o);
                cur[ps] += tot;
            } else {
                for (int q = 0; q < Wp; ++q) {
                    const uint32_t wq = (uint32_t)(ps * Wp + q);
                    if (wq >= W) break;
                    // cursor of worker wq lives in the lanes of group q
                    uint32_t c = __shfl_sync(0xFFFFFFFFu, cur[ps], q * E);
                    while (true) {
                        const uint32_t pp = c + (uint32_t)lane;
                        uint32_t ix2 = 0xFFFFFFFFu;
                        float v2 = 0.f;
                        if (pp < cnt) { ix2 = __ldg(ls.idx[wq] + pp); v2 = __ldg(ls.val[wq] + pp); }
                        const bool in2 = ix2 < hi;
                        if (in2) {
                            if (ix2 >= lo) tilebuf[ix2 - lo] = __fadd_rn(tilebuf[ix2 - lo], v2);
                            else record_status(hdr, -1 /*GC_E_INVALID*/, pp);
                        }
                        const unsigned m = __ballot_sync(0xFFFFFFFFu, in2);
                        c += (uint32_t)__popc(m);
                        __syncwarp();
                        if (m != 0xFFFFFFFFu) break;
                    }
                    if (lane / E == q) cur[ps] = c;
                }
            }
        }
        __syncwarp();
        // the tile leaves shared memory
        if (full && use_bulk) {
            if (lane == 0) bulk_store_tile(out + lo, tilebuf, (uint32_t)(kDecTile * sizeof(float)));
            __syncwarp();
        } else {
            for (uint32_t q = lane; q < hi - lo; q += 32) out[lo + q] = tilebuf[q];
            __syncwarp();
        }
    }
    if (t1 == ntl) {
        // the warp that owns the last tile: anything left in a list points at or beyond total_n
        for (int ps = 0; ps < passes; ++ps) {
            const uint32_t w = (uint32_t)(ps * Wp + lane / E);
            if (w < W && sub == 0 && cur[ps] < cnt) record_status(hdr, -1 /*GC_E_INVALID*/, cur[ps]);
        }
    }
    if (use_bulk && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

}  // namespace gc
