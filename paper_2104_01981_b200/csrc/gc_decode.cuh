// Tiled decode: dense_out = (zero | dense_out) + sum over workers of their sparse sets, with the
// additions applied in worker order 0..W-1 for every element (bit-reproducible).
//
// Every CTA owns a contiguous run of 8192-element tiles of the dense buffer.  A tile is built
// in shared memory -- cleared or loaded, then the entries of each worker that fall inside it
// are added, one worker after the other -- and leaves as one 32 KB bulk asynchronous copy
// (shared -> global) that overlaps with the building of the next tile in a second buffer, so
// the dense buffer is written exactly once, fully coalesced, and never read in zero-first mode.
// Each worker's list is sorted by index, so the CTA walks it with a
// cursor; the cursors' starting points are found once per CTA by a 32-way search per worker.
// The threads are split evenly among the workers and pre-load the next few entries of every
// worker at once, so a tile costs one round trip to the lists whatever W is.
#pragma once
#include "gc_common.cuh"

namespace gc {

constexpr int kDecTile = 8192;               // floats per CTA tile
constexpr int kDecBlock = 256;
constexpr int kDecRounds = 4;                // entries a thread pre-loads per tile
constexpr size_t kDecWideEntries = 4096;     // ring entries (8 bytes each) the wide kernel keeps in shared memory, all workers together
constexpr size_t kDecTileBytes = kDecTile * sizeof(float);

struct DecodeLists {
    const uint32_t* idx[64];
    const float* val[64];
    const uint32_t* len[64];     // device: number of valid pairs of the list (its first word), or null = `cnt`
};

// Starts the copy of one finished tile to global memory and returns at once; the tile buffer
// may be rewritten only after bulk_wait_read<N>() has shown that this copy has read it.
__device__ __forceinline__ void bulk_store_tile(float* gdst, const float* ssrc, uint32_t bytes) {
    // generic-proxy writes to shared memory must be fenced before the async proxy reads them
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    const uint32_t sa = (uint32_t)__cvta_generic_to_shared(ssrc);
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(gdst), "r"(sa), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Waits until all but the N most recent bulk copies of this thread have finished reading
// their shared-memory source.
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

// First position p in idx[0..cnt) with idx[p] >= key; all 32 lanes of a warp cooperate
// (33-way split per round, about four rounds for a million entries).
__device__ __forceinline__ uint32_t warp_lower_bound(const uint32_t* __restrict__ idx, uint32_t cnt,
                                                     uint32_t key, int lane) {
    uint32_t lo = 0, hi = cnt;                           // answer in [lo, hi]
    while (hi > lo) {
        const uint32_t span = hi - lo;
        const uint32_t p = lo + (uint32_t)(((unsigned long long)span * (uint32_t)(lane + 1)) / 33u);   // < hi
        const bool ge = __ldg(idx + p) >= key;           // monotone over the lanes
        const unsigned b = __ballot_sync(0xFFFFFFFFu, ge);
        // first lane that saw >= key bounds hi, the lane before it bounds lo
        const int f = b ? (__ffs(b) - 1) : 32;
        const uint32_t pf = lo + (uint32_t)(((unsigned long long)span * (uint32_t)(f + 1)) / 33u);
        const uint32_t pl = lo + (uint32_t)(((unsigned long long)span * (uint32_t)f) / 33u);
        const uint32_t nlo = f > 0 ? pl + 1 : lo;
        const uint32_t nhi = f < 32 ? pf : hi;
        lo = nlo; hi = nhi < nlo ? nlo : nhi;
    }
    return lo;
}

// Optimizer fused behind the decode (APPLY): the summed tile never goes to memory; it is scaled
// and fed to momentum SGD, v' = mu v + scale * sum, p' = p - lr v', on the parameter and velocity
// tiles read from and written back to global memory.
struct ApplyArgs {
    float* param;
    float* vel;
    float lr, mu, scale;
};

// The optimizer step on one finished tile: the sum stays on chip, parameter and velocity tiles
// stream through registers.
__device__ __forceinline__ void apply_tile(const ApplyArgs& ap, const float* s_tile, uint32_t lo, uint32_t hi,
                                           bool full, int tid) {
    if (full) {
#pragma unroll
        for (int q = 0; q < kDecTile / (4 * kDecBlock); ++q) {
            const uint32_t e4 = (uint32_t)(q * kDecBlock + tid);
            const float4 gs = *reinterpret_cast<const float4*>(s_tile + e4 * 4);
            float4 vv = __ldcs(reinterpret_cast<const float4*>(ap.vel + lo) + e4);
            float4 pp = __ldcs(reinterpret_cast<const float4*>(ap.param + lo) + e4);
            vv.x = __fadd_rn(__fmul_rn(ap.mu, vv.x), __fmul_rn(ap.scale, gs.x));
            vv.y = __fadd_rn(__fmul_rn(ap.mu, vv.y), __fmul_rn(ap.scale, gs.y));
            vv.z = __fadd_rn(__fmul_rn(ap.mu, vv.z), __fmul_rn(ap.scale, gs.z));
            vv.w = __fadd_rn(__fmul_rn(ap.mu, vv.w), __fmul_rn(ap.scale, gs.w));
            pp.x = __fsub_rn(pp.x, __fmul_rn(ap.lr, vv.x)); pp.y = __fsub_rn(pp.y, __fmul_rn(ap.lr, vv.y));
            pp.z = __fsub_rn(pp.z, __fmul_rn(ap.lr, vv.z)); pp.w = __fsub_rn(pp.w, __fmul_rn(ap.lr, vv.w));
            __stcs(reinterpret_cast<float4*>(ap.vel + lo) + e4, vv);
            __stcs(reinterpret_cast<float4*>(ap.param + lo) + e4, pp);
        }
    } else {
        for (uint32_t q = tid; q < hi - lo; q += kDecBlock) {
            const float vn = __fadd_rn(__fmul_rn(ap.mu, ap.vel[lo + q]), __fmul_rn(ap.scale, s_tile[q]));
            ap.vel[lo + q] = vn;
            ap.param[lo + q] = __fsub_rn(ap.param[lo + q], __fmul_rn(ap.lr, vn));
        }
    }
}

// Clears the tile, or loads it from the dense buffer when the sum continues what is there.
__device__ __forceinline__ void stage_tile(float* s_tile, const float* out, uint32_t lo, uint32_t hi, bool full,
                                           int zero_first, int use_bulk, int tid) {
    if (zero_first) {
#pragma unroll
        for (int q = 0; q < kDecTile / (4 * kDecBlock); ++q)
            *reinterpret_cast<float4*>(s_tile + (q * kDecBlock + tid) * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
    } else if (full && use_bulk) {
#pragma unroll
        for (int q = 0; q < kDecTile / (4 * kDecBlock); ++q)
            *reinterpret_cast<float4*>(s_tile + (q * kDecBlock + tid) * 4) =
                *reinterpret_cast<const float4*>(out + lo + (q * kDecBlock + tid) * 4);
    } else {
        for (uint32_t q = tid; q < (uint32_t)kDecTile; q += kDecBlock) s_tile[q] = (lo + q < hi) ? out[lo + q] : 0.f;
    }
}

// Counted route of the narrow kernels, for tiles that start at +0 and enough workers that their
// W block-wide steps would cost more than this.  Every pre-loaded entry inside [seg_lo, seg_hi)
// first counts itself into its element -- the tile doubles as the counter array -- which tells
// how many workers hit the element and gives each hitter a distinct arrival number.  One hit:
// the entry is stored.  Two hits: the first arrival stores, the second adds; fp32 addition is
// commutative, so (+0 + a) + b is the worker-order result whichever came first.  Three or more:
// there the order matters; those entries go to a short list and one thread per element sums
// them by worker number.  Returns false when the list overflowed: the touched elements are
// back at +0 and the caller applies the entries on the ordered route.  Called by the whole CTA.
constexpr uint32_t kDecCountedFrom = 4;      // workers from which the counted route is taken
constexpr int kDecConfCap = 128;             // colliding entries (three and more hits) a tile may hold
template <int R>
__device__ __forceinline__ bool counted_apply(float* s_tile, uint32_t lo, uint32_t seg_lo, uint32_t seg_hi,
                                              uint32_t (&ix)[R], const float (&v)[R], uint32_t my_w,
                                              uint32_t c0, WsHeader* hdr, uint4* s_conf, uint32_t* s_nconf, int tid) {
    int* const t_cnt = reinterpret_cast<int*>(s_tile);
    // per entry one byte: arrival number (6 bits) | min(hits, 3) << 6.  Four entries: a register
    // each (packing them cost registers and 5 % of the time); eight entries: packed into 64 bits,
    // which keeps that form at 64 registers and four CTAs per SM.
    constexpr bool kPacked = R > 4;
    uint32_t oh_a[kPacked ? 1 : R] = {};
    unsigned long long oh_p = 0ull;
    auto put = [&](int rd, uint32_t bits) { if constexpr (kPacked) oh_p |= (unsigned long long)bits << (8 * rd); else oh_a[rd] |= bits; };
    auto get = [&](int rd) -> uint32_t { if constexpr (kPacked) return (uint32_t)(oh_p >> (8 * rd)) & 255u; else return oh_a[rd]; };
#pragma unroll
    for (int rd = 0; rd < R; ++rd) {
        if (ix[rd] < seg_hi) {
            if (ix[rd] >= seg_lo) put(rd, (uint32_t)atomicAdd(&t_cnt[ix[rd] - lo], 1) & 63u);
            else { record_status(hdr, -1 /*GC_E_INVALID*/, c0); ix[rd] = 0xFFFFFFFFu; }     // list not ascending: skipped
        }
    }
    __syncthreads();
#pragma unroll
    for (int rd = 0; rd < R; ++rd)
        if (ix[rd] < seg_hi) put(rd, min((uint32_t)t_cnt[ix[rd] - lo], 3u) << 6);
    __syncthreads();                                       // every count has been read
    bool conflict = false;
#pragma unroll
    for (int rd = 0; rd < R; ++rd) {
        if (ix[rd] >= seg_hi) continue;
        const uint32_t b8 = get(rd);
        if ((b8 >> 6) <= 2u) {
            if ((b8 & 63u) == 0u) s_tile[ix[rd] - lo] = __fadd_rn(0.0f, v[rd]);
        } else {
            const uint32_t slot = atomicAdd(s_nconf, 1u);
            if (slot < (uint32_t)kDecConfCap) s_conf[slot] = make_uint4(ix[rd] - lo, my_w, __float_as_uint(v[rd]), 0u);
            conflict = true;
        }
    }
    bool done = true;
    if (__syncthreads_or(conflict ? 1 : 0)) {
        const uint32_t nc = *s_nconf;
        if (nc > (uint32_t)kDecConfCap) {
            // more colliding entries than the list holds: every touched element goes back to +0
            __syncthreads();
#pragma unroll
            for (int rd = 0; rd < R; ++rd) if (ix[rd] < seg_hi) s_tile[ix[rd] - lo] = 0.0f;
            done = false;
        } else if ((uint32_t)tid < nc) {
            // one thread per element with three or more hits: the entry of the lowest worker sums them all
            const uint4 me = s_conf[tid];
            bool lowest = true;
            for (uint32_t j = 0; j < nc; ++j) lowest = lowest && !(s_conf[j].x == me.x && s_conf[j].y < me.y);
            if (lowest) {
                float sum = 0.0f;
                uint32_t next_from = 0u;                   // workers below this one have been added
                while (true) {
                    uint32_t best = 0xFFFFFFFFu, bj = 0;
                    for (uint32_t j = 0; j < nc; ++j) {
                        const uint4 e = s_conf[j];
                        if (e.x == me.x && e.y >= next_from && e.y < best) { best = e.y; bj = j; }
                    }
                    if (best == 0xFFFFFFFFu) break;
                    sum = __fadd_rn(sum, __uint_as_float(s_conf[bj].z));
                    next_from = best + 1u;
                }
                s_tile[me.x] = sum;
            }
        }
    }
    if (done) {
#pragma unroll
        for (int rd = 0; rd < R; ++rd)
            if (ix[rd] < seg_hi && get(rd) == ((2u << 6) | 1u))
                s_tile[ix[rd] - lo] = __fadd_rn(s_tile[ix[rd] - lo], v[rd]);
    }
    __syncthreads();
    return done;
}

// R = entries a thread pre-loads per tile (R, or twice that for lists that are denser
// than four per thread and worker but still fit eight).
template <bool APPLY, int R>
// (the eight-entry form is held to 64 registers: four CTAs per SM measured better than three;
// holding the four-entry form to 40 registers for six CTAs per SM measured worse than five)
static __global__ void __launch_bounds__(kDecBlock, R == kDecRounds ? 0 : 4)
k_decode_tiles(DecodeLists ls, uint32_t W, uint32_t cnt, uint32_t total_n, float* __restrict__ out,
               int zero_first, int use_bulk, int nbuf, WsHeader* hdr, ApplyArgs ap) {
    // nbuf tile buffers: with two, one fills while the other drains (pays off when there are few
    // workers per tile; with many workers more resident CTAs are worth more than the overlap)
    extern __shared__ __align__(128) float s_tiles[];
    __shared__ uint32_t s_cur[64], s_len[64], s_nconf;
    __shared__ uint4 s_conf[kDecConfCap];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t ntl = (total_n + kDecTile - 1) / kDecTile;
    const uint32_t per = (ntl + gridDim.x - 1) / gridDim.x;
    const uint32_t t0 = blockIdx.x * per, t1 = min(ntl, t0 + per);
    if (t0 >= t1) return;

    // length of each worker's list, and where it enters this CTA's run of tiles
    for (uint32_t w = warp; w < W; w += kDecBlock / 32) {
        const uint32_t len = ls.len[w] != nullptr ? min(__ldg(ls.len[w]), cnt) : cnt;
        const uint32_t c = warp_lower_bound(ls.idx[w], len, t0 * (uint32_t)kDecTile, lane);
        if (lane == 0) { s_cur[w] = c; s_len[w] = len; }
    }
    // E consecutive threads serve one worker; passes of Wp workers cover W > 256 / E
    int Wp = 1;
    while (Wp < (int)W && Wp < 64) Wp <<= 1;
    const int E = kDecBlock / Wp;                        // 256 (W = 1) ... 4 (W = 64)
    const uint32_t my_w = (uint32_t)(tid / E);
    const int sub = tid % E;
    const bool live = my_w < W;
    __syncthreads();
    const uint32_t my_len = live ? s_len[my_w] : 0u;

    for (uint32_t tl = t0; tl < t1; ++tl) {
        float* const s_tile = s_tiles + (nbuf == 2 ? ((tl - t0) & 1u) : 0u) * kDecTile;
        if (use_bulk) {                                  // the copy that last used this buffer must have read it
            if (tid == 0) { if (nbuf == 2) bulk_wait_read<1>(); else bulk_wait_read<0>(); }
            __syncthreads();
        }
        const uint32_t lo = tl * (uint32_t)kDecTile;
        const uint32_t hi = min(total_n, lo + (uint32_t)kDecTile);
        const bool full = hi - lo == (uint32_t)kDecTile;
        stage_tile(s_tile, out, lo, hi, full, zero_first, use_bulk, tid);
        // pre-load the next R * E entries of every worker
        const uint32_t c0 = live ? s_cur[my_w] : 0u;
        uint32_t ix[R];
        float v[R];
        uint32_t nin = 0;
#pragma unroll
        for (int rd = 0; rd < R; ++rd) {
            const uint32_t p = c0 + (uint32_t)(rd * E + sub);
            ix[rd] = 0xFFFFFFFFu; v[rd] = 0.f;
            if (live && p < my_len) { ix[rd] = __ldg(ls.idx[my_w] + p); v[rd] = __ldg(ls.val[my_w] + p); }
        }
#pragma unroll
        for (int rd = 0; rd < R; ++rd) nin += ix[rd] < hi;       // sorted lists: the ins are a prefix
        // a worker whose pre-loaded entries all fall inside may have more: then the tile takes
        // the strictly sequential path so that worker order is kept for every element
        const bool maybe_more = (ix[R - 1] < hi) && sub == E - 1;
        if (tid == 0) s_nconf = 0u;
        if (!__syncthreads_or(maybe_more ? 1 : 0)) {                      // (also: tile staged, cursors read)
            const bool counted = zero_first && W >= kDecCountedFrom &&
                                 counted_apply<R>(s_tile, lo, lo, hi, ix, v, my_w, c0, hdr, s_conf, &s_nconf, tid);
            for (uint32_t q = 0; q < W && !counted; ++q) {                 // apply in worker order
                if (my_w == q) {
#pragma unroll
                    for (int rd = 0; rd < R; ++rd) {
                        if (ix[rd] < hi) {
                            if (ix[rd] >= lo) s_tile[ix[rd] - lo] = __fadd_rn(s_tile[ix[rd] - lo], v[rd]);
                            else record_status(hdr, -1 /*GC_E_INVALID*/, c0);      // list not ascending
                        }
                    }
                }
                __syncthreads();
            }
            if (live && nin) atomicAdd(&s_cur[my_w], nin);
        } else {
            for (uint32_t q = 0; q < W; ++q) {
                uint32_t c = s_cur[q];
                const uint32_t qlen = s_len[q];
                __syncthreads();
                while (true) {
                    const uint32_t pp = c + (uint32_t)tid;
                    uint32_t ix2 = 0xFFFFFFFFu;
                    float v2 = 0.f;
                    if (pp < qlen) { ix2 = __ldg(ls.idx[q] + pp); v2 = __ldg(ls.val[q] + pp); }
                    const bool in2 = ix2 < hi;
                    if (in2) {
                        if (ix2 >= lo) s_tile[ix2 - lo] = __fadd_rn(s_tile[ix2 - lo], v2);
                        else record_status(hdr, -1 /*GC_E_INVALID*/, pp);
                    }
                    const int m = __syncthreads_count(in2 ? 1 : 0);
                    c += (uint32_t)m;
                    if (m != kDecBlock) break;
                }
                if (tid == 0) s_cur[q] = c;
            }
        }
        __syncthreads();
        if (APPLY) {
            apply_tile(ap, s_tile, lo, hi, full, tid);
            __syncthreads();
            continue;
        }
        // the tile leaves shared memory
        if (full && use_bulk) {
            if (tid == 0) bulk_store_tile(out + lo, s_tile, (uint32_t)(kDecTile * sizeof(float)));
        } else {
            for (uint32_t q = tid; q < hi - lo; q += kDecBlock) out[lo + q] = s_tile[q];
        }
        __syncthreads();
    }
    if (t1 == ntl && tid < (int)W && s_cur[tid] < s_len[tid])
        record_status(hdr, -1 /*GC_E_INVALID*/, s_cur[tid]);   // leftovers point at or beyond total_n
    if (use_bulk && tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// Tiled decode of lists that carry per-tensor counts (threshold mode, plans of several tensors):
// worker w's pairs of tensor t sit in slots [out_off_t, out_off_t + count_w[t]) and the slots up
// to the tensor's capacity are unused, so a list is ascending only inside a tensor.  The tile
// loop of k_decode_tiles is kept (staged tile, workers applied in order, one bulk copy out); a
// tile is cut into segments at the tensor boundaries that fall inside it, and whenever the CTA
// moves on to the next tensor every worker's cursor jumps to that tensor's first slot and its
// end becomes that tensor's count.  Tiles inside one tensor (nearly all of them) cost what they
// cost in k_decode_tiles; a boundary costs one more round trip for the counts.
template <bool APPLY>
static __global__ void __launch_bounds__(kDecBlock)
k_decode_segments(DecodeLists ls, uint32_t W, const TensorDesc* __restrict__ desc, uint32_t T,
                  const uint32_t* __restrict__ tile_tensor, uint32_t total_n, float* __restrict__ out, int zero_first, int use_bulk, int nbuf, WsHeader* hdr, ApplyArgs ap) {
    extern __shared__ __align__(128) float s_tiles[];
    __shared__ uint32_t s_cur[64], s_len[64], s_nconf;
    __shared__ uint4 s_conf[kDecConfCap];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t ntl = (total_n + kDecTile - 1) / kDecTile;
    const uint32_t per = (ntl + gridDim.x - 1) / gridDim.x;
    const uint32_t t0 = blockIdx.x * per, t1 = min(ntl, t0 + per);
    if (t0 >= t1) return;

    // the tensor that holds the first element of this CTA's run (a table the plan made: one load
    // instead of a binary search over the tensor table in front of every CTA's first tile)
    uint32_t ct = __ldg(tile_tensor + t0);
    uint32_t d_end = __ldg(&desc[ct].off) + __ldg(&desc[ct].n);       // one past the tensor's last element
    uint32_t d_out = __ldg(&desc[ct].out_off), d_cap = __ldg(&desc[ct].cap);
    for (uint32_t w = warp; w < W; w += kDecBlock / 32) {
        const uint32_t m = min(__ldg(ls.len[w] + ct), d_cap);
        const uint32_t c = warp_lower_bound(ls.idx[w] + d_out, m, t0 * (uint32_t)kDecTile, lane);
        if (lane == 0) { s_cur[w] = d_out + c; s_len[w] = d_out + m; }
    }
    int Wp = 1;
    while (Wp < (int)W && Wp < 64) Wp <<= 1;
    const int E = kDecBlock / Wp;
    const uint32_t my_w = (uint32_t)(tid / E);
    const int sub = tid % E;
    const bool live = my_w < W;
    __syncthreads();

    for (uint32_t tl = t0; tl < t1; ++tl) {
        float* const s_tile = s_tiles + (nbuf == 2 ? ((tl - t0) & 1u) : 0u) * kDecTile;
        if (use_bulk) {                                  // the copy that last used this buffer must have read it
            if (tid == 0) { if (nbuf == 2) bulk_wait_read<1>(); else bulk_wait_read<0>(); }
            __syncthreads();
        }
        const uint32_t lo = tl * (uint32_t)kDecTile;
        const uint32_t hi = min(total_n, lo + (uint32_t)kDecTile);
        const bool full = hi - lo == (uint32_t)kDecTile;
        stage_tile(s_tile, out, lo, hi, full, zero_first, use_bulk, tid);
        uint32_t seg_lo = lo;
        while (true) {
            const uint32_t seg_hi = min(hi, d_end);
            const uint32_t my_len = live ? s_len[my_w] : 0u;
            const uint32_t c0 = live ? s_cur[my_w] : 0u;
            // the tensor ends inside this tile: the next tensor's table entry and this worker's count
            // for it are fetched together with the list entries (one round trip for both)
            const bool ends = d_end <= hi && ct + 1u < T;
            uint32_t nn = 0, n_off = 0, n_out = 0, n_cap = 0, ncnt = 0;
            if (ends) {
                nn = __ldg(&desc[ct + 1u].n); n_off = __ldg(&desc[ct + 1u].off);
                n_out = __ldg(&desc[ct + 1u].out_off); n_cap = __ldg(&desc[ct + 1u].cap);
                if (tid < (int)W) ncnt = __ldg(ls.len[tid] + ct + 1u);
            }
            uint32_t ix[kDecRounds];
            float v[kDecRounds];
            uint32_t nin = 0;
#pragma unroll
            for (int rd = 0; rd < kDecRounds; ++rd) {
                const uint32_t p = c0 + (uint32_t)(rd * E + sub);
                ix[rd] = 0xFFFFFFFFu; v[rd] = 0.f;
                if (live && p < my_len) { ix[rd] = __ldg(ls.idx[my_w] + p); v[rd] = __ldg(ls.val[my_w] + p); }
            }
#pragma unroll
            for (int rd = 0; rd < kDecRounds; ++rd) nin += ix[rd] < seg_hi;
            const bool maybe_more = (ix[kDecRounds - 1] < seg_hi) && sub == E - 1;
            if (tid == 0) s_nconf = 0u;
            if (!__syncthreads_or(maybe_more ? 1 : 0)) {                  // (also: tile staged, cursors read)
                const bool counted = zero_first && W >= kDecCountedFrom &&
                                     counted_apply<kDecRounds>(s_tile, lo, seg_lo, seg_hi, ix, v, my_w, c0, hdr, s_conf, &s_nconf, tid);
                for (uint32_t q = 0; q < W && !counted; ++q) {             // apply in worker order
                    if (my_w == q) {
#pragma unroll
                        for (int rd = 0; rd < kDecRounds; ++rd) {
                            if (ix[rd] < seg_hi) {
                                if (ix[rd] >= seg_lo) s_tile[ix[rd] - lo] = __fadd_rn(s_tile[ix[rd] - lo], v[rd]);
                                else record_status(hdr, -1 /*GC_E_INVALID*/, c0);      // not ascending / outside its tensor
                            }
                        }
                    }
                    __syncthreads();
                }
                if (live && nin) atomicAdd(&s_cur[my_w], nin);
            } else {
                for (uint32_t q = 0; q < W; ++q) {
                    uint32_t c = s_cur[q];
                    const uint32_t qlen = s_len[q];
                    __syncthreads();
                    while (true) {
                        const uint32_t pp = c + (uint32_t)tid;
                        uint32_t ix2 = 0xFFFFFFFFu;
                        float v2 = 0.f;
                        if (pp < qlen) { ix2 = __ldg(ls.idx[q] + pp); v2 = __ldg(ls.val[q] + pp); }
                        const bool in2 = ix2 < seg_hi;
                        if (in2) {
                            if (ix2 >= seg_lo) s_tile[ix2 - lo] = __fadd_rn(s_tile[ix2 - lo], v2);
                            else record_status(hdr, -1 /*GC_E_INVALID*/, pp);
                        }
                        const int m = __syncthreads_count(in2 ? 1 : 0);
                        c += (uint32_t)m;
                        if (m != kDecBlock) break;
                    }
                    if (tid == 0) s_cur[q] = c;
                }
            }
            __syncthreads();
            if (seg_hi < d_end) break;                   // the tile ends inside the tensor
            // the tensor ends here: whatever a list still holds for it points beyond its end
            if (tid < (int)W && s_cur[tid] < s_len[tid]) record_status(hdr, -1 /*GC_E_INVALID*/, s_cur[tid]);
            ++ct;
            while (ct < T && nn == 0u) {                  // (tensors without elements are stepped over)
                if (++ct >= T) break;
                nn = __ldg(&desc[ct].n); n_off = __ldg(&desc[ct].off);
                n_out = __ldg(&desc[ct].out_off); n_cap = __ldg(&desc[ct].cap);
                if (tid < (int)W) ncnt = __ldg(ls.len[tid] + ct);
            }
            if (ct >= T) { d_end = 0xFFFFFFFFu; break; }  // (only after the last element of the buffer)
            d_end = n_off + nn; d_out = n_out; d_cap = n_cap;
            if (tid < (int)W) { s_cur[tid] = d_out; s_len[tid] = d_out + min(ncnt, d_cap); }   // (own entries only)
            __syncthreads();
            if (seg_hi >= hi) break;                     // the tensor ended together with the tile
            seg_lo = seg_hi;
        }
        if (APPLY) {
            apply_tile(ap, s_tile, lo, hi, full, tid);
            __syncthreads();
            continue;
        }
        if (full && use_bulk) {
            if (tid == 0) bulk_store_tile(out + lo, s_tile, (uint32_t)(kDecTile * sizeof(float)));
        } else {
            for (uint32_t q = tid; q < hi - lo; q += kDecBlock) out[lo + q] = s_tile[q];
        }
        __syncthreads();
    }
    if (use_bulk && tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// 4-byte asynchronous copy global -> shared, and the wait for all such copies of this thread.
__device__ __forceinline__ void cp_async_4(void* sdst, const void* gsrc) {
    const uint32_t sa = (uint32_t)__cvta_generic_to_shared(sdst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(sa), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Decode for many workers or dense lists.  Every worker's next `win` entries sit in a ring in
// shared memory that is topped up with asynchronous copies as entries are consumed, so every
// list entry is fetched once and the fetch for the next tile overlaps with this tile's way out.
// The workers are applied one after the other, each by the whole CTA (one ring entry per
// thread), so a worker's share of a tile may be as large as the ring whatever the number of
// workers, and the block-wide count that separates two workers also yields how far the cursor
// moves.  If some worker has more than `win` entries in the tile, the pass ends at the smallest
// index up to which every worker's ring is complete and the rest of the tile takes another
// pass.  One tile buffer; `win` is a power of two.
template <bool APPLY>
static __global__ void __launch_bounds__(kDecBlock)
k_decode_wide(DecodeLists ls, uint32_t W, uint32_t cnt, uint32_t total_n, float* __restrict__ out,
              int zero_first, int use_bulk, uint32_t win, WsHeader* hdr, ApplyArgs ap) {
    extern __shared__ __align__(128) float s_tiles[];
    float* const s_tile = s_tiles;
    uint32_t* const rg_idx = reinterpret_cast<uint32_t*>(s_tiles + kDecTile);      // [W][win]
    float* const rg_val = reinterpret_cast<float*>(rg_idx + W * win);              // [W][win]
    __shared__ uint32_t s_cur[64], s_len[64], s_adv[64], s_bound;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t ntl = (total_n + kDecTile - 1) / kDecTile;
    const uint32_t per = (ntl + gridDim.x - 1) / gridDim.x;
    const uint32_t t0 = blockIdx.x * per, t1 = min(ntl, t0 + per);
    if (t0 >= t1) return;
    const uint32_t mask = win - 1u;
    // E consecutive threads top up one worker's ring
    int Wp = 1;
    while (Wp < (int)W && Wp < 64) Wp <<= 1;
    const int E = kDecBlock / Wp;
    const uint32_t my_w = (uint32_t)(tid / E);
    const int sub = tid % E;

    for (uint32_t w = warp; w < W; w += kDecBlock / 32) {
        const uint32_t len = ls.len[w] != nullptr ? min(__ldg(ls.len[w]), cnt) : cnt;
        const uint32_t c = warp_lower_bound(ls.idx[w], len, t0 * (uint32_t)kDecTile, lane);
        if (lane == 0) { s_cur[w] = c; s_len[w] = len; s_adv[w] = 0u; }
    }
    __syncthreads();
    // list positions [from, to) of worker my_w go to their ring slots
    auto top_up = [&](uint32_t from, uint32_t to) {
        for (uint32_t p = from + (uint32_t)sub; p < to; p += (uint32_t)E) {
            cp_async_4(rg_idx + my_w * win + (p & mask), ls.idx[my_w] + p);
            cp_async_4(rg_val + my_w * win + (p & mask), ls.val[my_w] + p);
        }
    };
    if (my_w < W) top_up(s_cur[my_w], min(s_len[my_w], s_cur[my_w] + win));

    for (uint32_t tl = t0; tl < t1; ++tl) {
        const uint32_t lo = tl * (uint32_t)kDecTile;
        const uint32_t hi = min(total_n, lo + (uint32_t)kDecTile);
        const bool full = hi - lo == (uint32_t)kDecTile;
        if (use_bulk && !APPLY && tid == 0) bulk_wait_read<0>();     // the previous tile has left the buffer
        cp_async_wait_all();
        if (tid == 0) s_bound = hi;
        __syncthreads();                                 // rings complete, cursors settled, buffer free
        stage_tile(s_tile, out, lo, hi, full, zero_first, use_bulk, tid);
        uint32_t sub_lo = lo;
        while (true) {
            // a worker whose ring is full and ends inside the tile may have more entries there
            if ((uint32_t)tid < W) {
                const uint32_t cur = s_cur[tid];
                if (s_len[tid] - cur >= win) {
                    const uint32_t last = rg_idx[tid * win + ((cur + win - 1u) & mask)];
                    if (last < hi) atomicMin(&s_bound, last + 1u);
                }
            }
            __syncthreads();                             // (also: the staged tile is visible)
            uint32_t bound = s_bound;
            if (bound <= sub_lo) {                       // no progress: a list is not ascending
                if (tid == 0) record_status(hdr, -1 /*GC_E_INVALID*/, sub_lo);
                bound = hi;
            }
            for (uint32_t q = 0; q < W; ++q) {           // worker order
                const uint32_t cur = s_cur[q];
                const uint32_t avail = min(s_len[q] - cur, win);
                uint32_t adv = 0;
                for (uint32_t i0 = 0; i0 < win; i0 += kDecBlock) {
                    const uint32_t i = i0 + (uint32_t)tid;
                    const uint32_t slot = q * win + ((cur + i) & mask);
                    const uint32_t ix = i < avail ? rg_idx[slot] : 0xFFFFFFFFu;
                    const bool in = ix < bound;
                    if (in) {
                        if (ix >= sub_lo) s_tile[ix - lo] = __fadd_rn(s_tile[ix - lo], rg_val[slot]);
                        else record_status(hdr, -1 /*GC_E_INVALID*/, ix);      // behind the cursor: skipped
                    }
                    const uint32_t c = (uint32_t)__syncthreads_count(in ? 1 : 0);   // next worker may start
                    adv += c;
                    if (c < (uint32_t)kDecBlock) break;                          // ascending: nothing more below the bound
                }
                if (tid == 0) { s_cur[q] = cur + adv; s_adv[q] = adv; }
            }
            if (tid == 0) s_bound = hi;
            __syncthreads();                             // cursors moved
            if (my_w < W) {                              // the consumed slots are topped up
                const uint32_t cur = s_cur[my_w], len = s_len[my_w];
                top_up(min(len, cur - s_adv[my_w] + win), min(len, cur + win));
            }
            if (bound >= hi) break;
            cp_async_wait_all();
            __syncthreads();
            sub_lo = bound;
        }
        if (APPLY) {
            apply_tile(ap, s_tile, lo, hi, full, tid);
            continue;                                    // (the barrier at the top of the loop orders the reuse)
        }
        if (full && use_bulk) {
            if (tid == 0) bulk_store_tile(out + lo, s_tile, (uint32_t)(kDecTile * sizeof(float)));
        } else {
            for (uint32_t q = tid; q < hi - lo; q += kDecBlock) out[lo + q] = s_tile[q];
        }
    }
    cp_async_wait_all();
    __syncthreads();
    if (t1 == ntl && tid < (int)W && s_cur[tid] < s_len[tid])
        record_status(hdr, -1 /*GC_E_INVALID*/, s_cur[tid]);   // leftovers point at or beyond total_n
    if (use_bulk && !APPLY && tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// Decode without a fixed order among the workers (GC_OPT_DECODE_ORDER = GC_ORDER_ANY): the rings
// of k_decode_wide, but all entries of a pass are added at once with shared-memory atomics, so
// a tile costs a constant number of block-wide steps whatever W is.  The sum of an element that
// several workers hit is then rounded in an order that may change from run to run: every result
// is within (hits - 1) x 2^-24 x sum |values| of the fixed-order one, and equal to it for
// elements hit once.
template <bool APPLY>
static __global__ void __launch_bounds__(kDecBlock)
k_decode_any(DecodeLists ls, uint32_t W, uint32_t cnt, uint32_t total_n, float* __restrict__ out,
             int zero_first, int use_bulk, uint32_t win, WsHeader* hdr, ApplyArgs ap) {
    extern __shared__ __align__(128) float s_tiles[];
    float* const s_tile = s_tiles;
    uint32_t* const rg_idx = reinterpret_cast<uint32_t*>(s_tiles + kDecTile);      // [W][win]
    float* const rg_val = reinterpret_cast<float*>(rg_idx + W * win);              // [W][win]
    __shared__ uint32_t s_cur[64], s_len[64], s_adv[64], s_bound;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t ntl = (total_n + kDecTile - 1) / kDecTile;
    const uint32_t per = (ntl + gridDim.x - 1) / gridDim.x;
    const uint32_t t0 = blockIdx.x * per, t1 = min(ntl, t0 + per);
    if (t0 >= t1) return;
    const uint32_t mask = win - 1u;
    // E consecutive threads serve one worker: they top up its ring and add its entries
    int Wp = 1;
    while (Wp < (int)W && Wp < 64) Wp <<= 1;
    const int E = kDecBlock / Wp;
    const uint32_t my_w = (uint32_t)(tid / E);
    const int sub = tid % E;

    for (uint32_t w = warp; w < W; w += kDecBlock / 32) {
        const uint32_t len = ls.len[w] != nullptr ? min(__ldg(ls.len[w]), cnt) : cnt;
        const uint32_t c = warp_lower_bound(ls.idx[w], len, t0 * (uint32_t)kDecTile, lane);
        if (lane == 0) { s_cur[w] = c; s_len[w] = len; s_adv[w] = 0u; }
    }
    __syncthreads();
    auto top_up = [&](uint32_t from, uint32_t to) {      // list positions [from, to) of worker my_w go to their ring slots
        for (uint32_t p = from + (uint32_t)sub; p < to; p += (uint32_t)E) {
            cp_async_4(rg_idx + my_w * win + (p & mask), ls.idx[my_w] + p);
            cp_async_4(rg_val + my_w * win + (p & mask), ls.val[my_w] + p);
        }
    };
    if (my_w < W) top_up(s_cur[my_w], min(s_len[my_w], s_cur[my_w] + win));

    for (uint32_t tl = t0; tl < t1; ++tl) {
        const uint32_t lo = tl * (uint32_t)kDecTile;
        const uint32_t hi = min(total_n, lo + (uint32_t)kDecTile);
        const bool full = hi - lo == (uint32_t)kDecTile;
        if (use_bulk && !APPLY && tid == 0) bulk_wait_read<0>();     // the previous tile has left the buffer
        cp_async_wait_all();
        if (tid == 0) s_bound = hi;
        __syncthreads();                                 // rings complete, cursors settled, buffer free
        stage_tile(s_tile, out, lo, hi, full, zero_first, use_bulk, tid);
        uint32_t sub_lo = lo;
        while (true) {
            if ((uint32_t)tid < W) {                     // a full ring that ends inside the tile may hide more entries
                const uint32_t cur = s_cur[tid];
                s_adv[tid] = 0u;
                if (s_len[tid] - cur >= win) {
                    const uint32_t last = rg_idx[tid * win + ((cur + win - 1u) & mask)];
                    if (last < hi) atomicMin(&s_bound, last + 1u);
                }
            }
            __syncthreads();                             // (also: the staged tile is visible)
            uint32_t bound = s_bound;
            if (bound <= sub_lo) {                       // no progress: a list is not ascending
                if (tid == 0) record_status(hdr, -1 /*GC_E_INVALID*/, sub_lo);
                bound = hi;
            }
            if (my_w < W) {
                const uint32_t cur = s_cur[my_w];
                const uint32_t avail = min(s_len[my_w] - cur, win);
                uint32_t below = 0;
                for (uint32_t i = (uint32_t)sub; i < avail; i += (uint32_t)E) {
                    const uint32_t slot = my_w * win + ((cur + i) & mask);
                    const uint32_t ix = rg_idx[slot];
                    if (ix >= bound) break;                                      // ascending: the rest lies above
                    ++below;
                    if (ix < sub_lo) { record_status(hdr, -1 /*GC_E_INVALID*/, ix); continue; }   // behind the cursor: skipped
                    atomicAdd(&s_tile[ix - lo], rg_val[slot]);
                }
                if (below) atomicAdd(&s_adv[my_w], below);
            }
            __syncthreads();                             // the tile is complete up to the bound
            if ((uint32_t)tid < W) s_cur[tid] += s_adv[tid];
            if (tid == 0) s_bound = hi;
            __syncthreads();                             // cursors moved
            if (my_w < W) {                              // the consumed slots are topped up
                const uint32_t nc = s_cur[my_w], len = s_len[my_w];
                top_up(min(len, nc - s_adv[my_w] + win), min(len, nc + win));
            }
            if (bound >= hi) break;
            cp_async_wait_all();
            __syncthreads();
            sub_lo = bound;
        }
        if (APPLY) {
            apply_tile(ap, s_tile, lo, hi, full, tid);
            continue;                                    // (the barrier at the top of the loop orders the reuse)
        }
        if (full && use_bulk) {
            if (tid == 0) bulk_store_tile(out + lo, s_tile, (uint32_t)(kDecTile * sizeof(float)));
        } else {
            for (uint32_t q = tid; q < hi - lo; q += kDecBlock) out[lo + q] = s_tile[q];
        }
    }
    cp_async_wait_all();
    __syncthreads();
    if (t1 == ntl && tid < (int)W && s_cur[tid] < s_len[tid])
        record_status(hdr, -1 /*GC_E_INVALID*/, s_cur[tid]);   // leftovers point at or beyond total_n
    if (use_bulk && !APPLY && tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

}  // namespace gc
