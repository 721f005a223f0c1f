// Shared device-side definitions of libgc: tensor table, workspace layout, tile geometry,
// warp/block scan helpers and the ordered-tile prefix exchange ("look-back").
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gc {

// ----------------------------------------------------------------------------- geometry
constexpr int kBlock = 256;                 // threads per CTA for the streaming kernels
constexpr int kWarps = kBlock / 32;
constexpr int kVpt = 4;                     // 128-bit vectors per thread per tile
constexpr int kTile = kBlock * kVpt * 4;    // 4096 elements per tile
constexpr int kWarpChunk = 32 * kVpt * 4;   // contiguous elements owned by one warp
constexpr int kSampleTile = kBlock;         // sample groups (of 4 elements) per sample tile: one per thread
constexpr uint32_t kKeyMask = 0x7FFFFFFFu;

// radix-select levels over the 31-bit magnitude key: 11 + 10 + 10 bits
constexpr int kLevels = 3;
__host__ __device__ constexpr int level_bits(int l) { return l == 0 ? 11 : 10; }
__host__ __device__ constexpr int level_shift(int l) { return l == 0 ? 20 : (l == 1 ? 10 : 0); }
__host__ __device__ constexpr bool level_is_first(int l) { return l == 0; }
constexpr int kHistBins = 2048;             // bins reserved per tensor (largest level)
constexpr int kSlab = 128;                  // candidate slots a warp reserves at a time

// Bounded waits: a predecessor tile is always already running (tiles are handed out by an
// atomic ticket), so these limits are a safety net, not a schedule.
constexpr uint32_t kSpinLimit = 1u << 21;

// ----------------------------------------------------------------------------- tables
struct TensorDesc {          // one per tensor, immutable, plan-owned device memory
    uint32_t off;            // first flat index
    uint32_t n;              // elements
    uint32_t k;              // entries to keep (top-k) / reference k (threshold)
    uint32_t cap;            // output capacity
    uint32_t out_off;        // first output slot
    uint32_t tile0;          // first tile id
    uint32_t ntiles;         // tiles of this tensor
    uint32_t stride;         // threshold mode: sampling stride in 4-element groups
    uint32_t sstride;        // stride (in 4-element groups) of the sample that sets the candidate
                             // threshold; 0 = tensor is not sampled, every element is a candidate
    uint32_t srank;          // rank taken inside the sample (k_s in threshold mode)
    uint32_t stile0;         // first sample tile id
    uint32_t nstiles;        // sample tiles (kSampleTile sample groups each)
    uint32_t group0;         // first compaction group id (a group = kWarps consecutive tiles)
    uint32_t ngroups;        // compaction groups of this tensor
    uint32_t kind;           // kKindRegular, or kKindSmall: the candidate path hands the whole tensor
                             // to one CTA that selects exactly on its own (no sample, no candidates)
    uint32_t pad;
};
constexpr uint32_t kKindRegular = 0u, kKindSmall = 1u;
constexpr uint32_t kSmallMax = kTile - 3;     // tensors below this many elements always lie inside one tile,
                                              // whatever their offset; "small" = fits one tile
static_assert(sizeof(TensorDesc) == 64, "tensor table entry is 64 bytes");

struct TensorSel {           // one per tensor, in the workspace, rewritten every call
    uint32_t prefix;         // key bits fixed so far by the radix select
    uint32_t krem;           // entries still to take inside the current prefix bucket
    uint32_t T;              // k-th largest key (valid after the last level)
    uint32_t m_eq;           // how many of the entries with key == T are taken
    uint32_t done[kLevels];  // tiles histogrammed per level
    uint32_t flags;          // kSelFailed: the candidate path gave up on this tensor
};
constexpr uint32_t kSelFailed = 1u;

struct WsHeader {            // head of the workspace, 256 bytes
    int32_t status;          // GC_OK / warning / error recorded by kernels
    uint32_t abort;          // non-zero: a bounded wait gave up, everyone leaves
    unsigned long long detail;
    uint32_t ticket[8];      // tile tickets, one per ordered kernel
    uint32_t cand_total;     // candidate slots handed out so far
    uint32_t overflow;       // candidate buffer ran out: every tensor takes the exact multi-pass path
    uint32_t n_failed;       // tensors whose candidate set turned out too small
    uint32_t barrier;        // arrivals at the grid barriers of the fused kernel (monotonic)
    uint32_t n_stamps;       // phase time stamps recorded by CTA 0 of the fused kernel
    uint32_t exit_count;     // CTAs of a fused top-k launch that have left (back to 0 when the last one leaves)
    uint32_t pad0[2];
    unsigned long long stamp[20];   // %globaltimer (ns) at the start and after each phase
    unsigned long long t_last_exit; // latest exit of any CTA of the fused kernel (ns)
    unsigned long long clean_mark;  // set by a fused top-k launch that left the control block clean (see CleanArgs)
};
// (as 32-bit words of the header: what those kernels do not reset at their start)
constexpr uint32_t kHdrBarrierWord = 15, kHdrExitWord = 17, kHdrSigWord = 62;
static_assert(sizeof(WsHeader) == 256, "header is 256 bytes");

struct WsView {              // host-computed pointers into the workspace
    WsHeader* hdr;
    TensorSel* sel;          // [n_tensors] selection record the kernel works on
    uint32_t* hist;          // [n_tensors][kHistBins]
    unsigned long long* tile_state;   // [ntiles] (or [ngroups]) look-back words
    const TensorSel* gate;   // non-null: only tensors the candidate path gave up on are processed
};

// Iteration spaces of the histogram kernels: every tile of a tensor, or its sample tiles.
struct FullSpace {
    __device__ static uint32_t tile0(const TensorDesc& d) { return d.tile0; }
    __device__ static uint32_t ntiles(const TensorDesc& d) { return d.ntiles; }
    __device__ static uint32_t rank(const TensorDesc& d) { return d.k; }
};
struct SampleSpace {
    __device__ static uint32_t tile0(const TensorDesc& d) { return d.stile0; }
    __device__ static uint32_t ntiles(const TensorDesc& d) { return d.nstiles; }
    __device__ static uint32_t rank(const TensorDesc& d) { return d.srank; }
};
struct GroupSpace {
    __device__ static uint32_t tile0(const TensorDesc& d) { return d.group0; }
    __device__ static uint32_t ntiles(const TensorDesc& d) { return d.ngroups; }
};

// ----------------------------------------------------------------------------- small helpers
__device__ __forceinline__ uint32_t key_of(float a) { return __float_as_uint(a) & kKeyMask; }

// Loads of data that another CTA may have written earlier in the SAME launch (the fused kernel
// runs all phases in one grid) must not be served from this SM's L1: read them at L2.
__device__ __forceinline__ uint32_t ld_cg(const uint32_t* p) { return __ldcg(p); }
__device__ __forceinline__ float ld_cg(const float* p) { return __ldcg(p); }
__device__ __forceinline__ float4 ld_cg(const float4* p) { return __ldcg(p); }
__device__ __forceinline__ uint2 ld_cg(const uint2* p) { return __ldcg(p); }
__device__ __forceinline__ uint4 ld_cg(const uint4* p) { return __ldcg(p); }
__device__ __forceinline__ unsigned long long ld_cg(const unsigned long long* p) { return __ldcg(p); }

// How the gradient is stored.  The kernels that read g are templates on one of these; the
// arithmetic is fp32 either way (a bf16 value is an fp32 value with 16 zero bits appended).
struct GradF32 {
    static __device__ __forceinline__ float ld1(const void* g, uint32_t i) {
        return __ldg(reinterpret_cast<const float*>(g) + i);
    }
    static __device__ __forceinline__ float4 ld4(const void* g, uint32_t i) {          // i a multiple of 4
        return __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(g) + i));
    }
    static __device__ __forceinline__ const void* at(const void* g, uint32_t i) {
        return reinterpret_cast<const float*>(g) + i;
    }
};
struct GradBF16 {
    static __device__ __forceinline__ float ld1(const void* g, uint32_t i) {
        return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(g) + i) << 16);
    }
    static __device__ __forceinline__ float4 ld4(const void* g, uint32_t i) {          // i a multiple of 4
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const unsigned short*>(g) + i));
        return make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xFFFF0000u),
                           __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xFFFF0000u));
    }
    static __device__ __forceinline__ const void* at(const void* g, uint32_t i) {
        return reinterpret_cast<const unsigned short*>(g) + i;
    }
};

constexpr int kEmitStage = 64;               // candidates of one warp chunk staged in shared memory

// Static shared memory of every streaming kernel (one instance per CTA, reused by all phases).
struct BlockSmem {
    uint32_t hist[2048];
    uint32_t scratch[kWarps + 4];
    uint32_t last, tile;
    uint32_t gt_tot[kWarps], eq_tot[kWarps], gt_ex[kWarps], eq_ex[kWarps];
    uint32_t gt_sum, eq_sum;
    unsigned long long excl;
    unsigned long long red[kWarps];
    int ok;
    uint2 emit[kWarps][kEmitStage];
};

__device__ __forceinline__ void record_status(WsHeader* h, int32_t code, unsigned long long detail) {
    // errors (negative) win over warnings; first writer of a kind keeps its detail
    int32_t old = atomicCAS(&h->status, 0, code);
    if (old == 0) { h->detail = detail; return; }
    if (old > 0 && code < 0) { atomicExch(&h->status, code); h->detail = detail; }
}

// Tensor that owns `tile` in iteration space S: the LAST t whose first tile is <= tile.
// Tensors without tiles share their first-tile id with their successor, so the last such t is
// the one that actually has tiles.
template <typename S = FullSpace>
__device__ __forceinline__ uint32_t find_tensor(const TensorDesc* __restrict__ d, uint32_t T, uint32_t tile) {
    uint32_t lo = 0, hi = T;                 // invariant: answer in [lo, hi)
    while (hi - lo > 1) {
        uint32_t mid = (lo + hi) >> 1;
        if (S::tile0(d[mid]) <= tile) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ bool gate_open(const WsView& ws, uint32_t t, const TensorDesc& d) {
    // with a gate, a tensor is processed only if the candidate path failed for it (or overall);
    // small tensors were finished by their own CTA and are never redone
    if (ws.gate == nullptr) return true;
    if (d.kind == kKindSmall) return false;
    return (ld_cg(&ws.gate[t].flags) & kSelFailed) != 0u || ld_cg(&ws.hdr->overflow) != 0u;
}
__device__ __forceinline__ bool nothing_to_redo(const WsView& ws) {
    return ws.gate != nullptr && ld_cg(&ws.hdr->n_failed) == 0u && ld_cg(&ws.hdr->overflow) == 0u;
}

struct TileGeom { uint32_t base, lo, hi; };  // aligned start, first and one-past-last valid flat index
__device__ __forceinline__ TileGeom tile_geom(const TensorDesc& d, uint32_t tile_in_tensor) {
    TileGeom g;
    g.base = (d.off & ~3u) + tile_in_tensor * (uint32_t)kTile;
    g.lo = max(d.off, g.base);
    uint32_t end = d.off + d.n;
    g.hi = min(end, g.base + (uint32_t)kTile);
    return g;
}

// flat index of element 0 of this thread's j-th vector inside a tile
__device__ __forceinline__ uint32_t vec_index(uint32_t base, int warp, int lane, int j) {
    return base + warp * kWarpChunk + (j * 32 + lane) * 4;
}

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t o = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}
__device__ __forceinline__ unsigned long long warp_incl_scan64(unsigned long long v, int lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}
__device__ __forceinline__ unsigned long long warp_sum64(unsigned long long v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}

// Per-thread counts c[j] (0..4) for its kVpt vectors -> exclusive rank of each vector within
// the warp's chunk in element order (vector j, then lane), plus the warp total.
// Counts are packed as 8-bit fields (a field never exceeds 32*4 = 128).
__device__ __forceinline__ void warp_rank(const uint32_t (&c)[kVpt], int lane,
                                          uint32_t (&rank)[kVpt], uint32_t& total) {
    uint32_t packed = 0;
#pragma unroll
    for (int j = 0; j < kVpt; ++j) packed |= c[j] << (8 * j);
    uint32_t incl = warp_incl_scan(packed, lane);
    uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
    uint32_t excl = incl - packed;
    uint32_t run = 0;
#pragma unroll
    for (int j = 0; j < kVpt; ++j) {
        rank[j] = run + ((excl >> (8 * j)) & 0xFFu);
        run += (tot >> (8 * j)) & 0xFFu;
    }
    total = run;
}

// Where the top-k kernels look for their sample (the sample only steers the candidate bracket;
// no result depends on it).  Sample group number sg -> 4-element group of the tensor: runs of
// eight consecutive groups, i.e. one 128-byte line, every 8 x sstride groups.  The same number
// of samples as one group every `sstride`, but an eighth of the scattered DRAM accesses -- the
// sample phase is bound by how many scattered reads per second the memory serves (about 24 G/s
// measured here), not by anything on the SM.  (The threshold variant's sample is part of its
// definition and stays one group every `stride`.)
__device__ __forceinline__ uint64_t sample_group(uint64_t sg, uint32_t sstride) {
    return (sg >> 3) * (8ull * sstride) + (sg & 7ull);
}

// One count per lane into a shared-memory histogram, aggregated over the warp first: lanes that
// hit the same bin elect one of them to add their number (keys of one tensor crowd into a
// handful of coarse bins, and 32 atomics on one shared-memory word are served one after the
// other).  bin = 0xFFFFFFFF: this lane has nothing to count.  All 32 lanes must call.
__device__ __forceinline__ void hist_add_warp(uint32_t* hist, uint32_t bin, int lane) {
    const unsigned peers = __match_any_sync(0xFFFFFFFFu, bin);
    if (bin != 0xFFFFFFFFu && (__ffs(peers) - 1) == lane) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
}

// ----------------------------------------------------------------------------- ordered tiles
// Tile descriptors: bits 63..62 = flag (0 none, 1 aggregate of this tile, 2 inclusive prefix
// up to and including this tile), bits 61..0 = value.  Flag and value travel in one 64-bit
// word, so a relaxed load sees a consistent pair.
constexpr unsigned long long kFlagAgg = 1ull << 62;
constexpr unsigned long long kFlagPre = 2ull << 62;
constexpr unsigned long long kValMask = (1ull << 62) - 1;

__device__ __forceinline__ unsigned long long ld_state(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_state(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}

// Called by all 32 lanes of one warp.  Publishes this tile's aggregate, walks back over the
// predecessor tiles of the same tensor until an inclusive prefix is met, publishes this
// tile's inclusive prefix and returns the exclusive one.  `ok` is cleared if a wait ran out
// (status GC_E_TIMEOUT recorded, abort raised).
__device__ __forceinline__ unsigned long long lookback(unsigned long long* state, uint32_t tile,
                                                       uint32_t first_tile, unsigned long long agg,
                                                       int lane, WsHeader* hdr, bool& ok) {
    ok = true;
    if (tile == first_tile) {
        if (lane == 0) st_state(state + tile, kFlagPre | agg);
        return 0ull;
    }
    if (lane == 0) st_state(state + tile, kFlagAgg | agg);
    unsigned long long excl = 0;
    long long base = (long long)tile - 1;
    while (true) {
        long long p = base - lane;
        unsigned long long v = kFlagPre;                 // before the tensor's first tile: prefix 0
        bool timed_out = false;
        if (p >= (long long)first_tile) {
            uint32_t spins = 0;
            v = ld_state(state + p);
            while ((v >> 62) == 0) {
                if (++spins > kSpinLimit) { timed_out = true; break; }
                if (spins > 16) __nanosleep(spins > 1024 ? 200 : 40);
                if ((spins & 1023u) == 0 && *(volatile uint32_t*)&hdr->abort) { timed_out = true; break; }
                v = ld_state(state + p);
            }
        }
        if (__any_sync(0xFFFFFFFFu, timed_out)) {
            if (lane == 0) {
                record_status(hdr, -5 /*GC_E_TIMEOUT*/, tile);
                atomicExch(&hdr->abort, 1u);
            }
            ok = false;
            return 0ull;
        }
        unsigned pmask = __ballot_sync(0xFFFFFFFFu, (v >> 62) == 2);
        int first_p = pmask ? (__ffs(pmask) - 1) : 32;
        unsigned long long contrib = (lane <= first_p) ? (v & kValMask) : 0ull;
        excl += warp_sum64(contrib);
        if (pmask) break;
        base -= 32;
    }
    if (lane == 0) st_state(state + tile, kFlagPre | ((excl + agg) & kValMask));
    return excl;
}

// Phase time stamp by CTA 0 (diagnostic).  The running index lives in a register of the caller
// so that the stamp is two stores and no load: a load here would sit on CTA 0's path to the
// next grid barrier, and every other CTA waits for that one.
__device__ __forceinline__ void phase_stamp(WsHeader* hdr, uint32_t& n, uint32_t b) {
    if (b == 0 && threadIdx.x == 0 && n < 20u) {
        unsigned long long ts;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ts));
        hdr->stamp[n] = ts;
        hdr->n_stamps = n + 1u;
    }
    ++n;
}

__device__ __forceinline__ void phase_stamp(WsHeader* hdr, uint32_t& n) { phase_stamp(hdr, n, blockIdx.x); }

__device__ __forceinline__ void exit_stamp(WsHeader* hdr) {
    if (threadIdx.x == 0) {
        unsigned long long ts;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ts));
        atomicMax(&hdr->t_last_exit, ts);
    }
}

// ----------------------------------------------------------------------------- grid barrier
// Barrier across the G CTAs that share one workspace header: all CTAs of a cooperative launch,
// or one of several independent groups inside it (all CTAs of the launch are resident either
// way).  The counter only grows: the b-th barrier waits for b * G arrivals.  The wait is
// bounded; if it runs out the abort flag is raised, GC_E_TIMEOUT is recorded and every CTA of
// the group leaves.
__device__ __forceinline__ bool grid_barrier(WsHeader* hdr, uint32_t& passed, int* s_ok, uint32_t G) {
    __syncthreads();
    if (threadIdx.x == 0) {
        int ok = 1;
        __threadfence();
        const uint32_t target = (passed + 1u) * G;
        atomicAdd(&hdr->barrier, 1u);
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
__device__ __forceinline__ bool grid_barrier(WsHeader* hdr, uint32_t& passed, int* s_ok) {
    return grid_barrier(hdr, passed, s_ok, gridDim.x);
}

// ----------------------------------------------------------------------------- a control block that stays clean
// The fused top-k kernels leave the control block of the workspace as their next launch needs to
// find it, so that launch can do without the clearing launch in front of it.  Everything that is
// first written after the first grid barrier is zeroed at the START of a launch, a slice per CTA
// (the writers come after the barrier, so there is no ordering problem); the sections written
// before the first barrier ("early": at most three ranges) are zeroed right after the barrier that
// follows their last reader; the barrier counter is reset by the CTA that leaves last (an exit
// counter in the header), which then sets a 64-bit mark.  When the host has skipped the clearing
// launch (on the caller's promise that nobody else writes to the workspace), the kernel first
// checks the mark and leaves at once if it is missing: no barrier is entered on a counter that
// cannot be trusted.  G CTAs share the block, this is CTA b of them.
struct CleanArgs {
    uint4* ctrl;                     // the control block (= the workspace), in 16-byte units
    uint32_t ctrl_units;             // its length
    uint32_t early[3][2];            // [begin, end) in units of the sections written before the first barrier
    unsigned long long mark;         // what the header's mark reads after a launch that left the block clean
    uint32_t expect_clean;           // the host skipped the clearing launch
};
__device__ __forceinline__ unsigned long long* clean_mark_ptr(WsHeader* hdr) {
    return reinterpret_cast<unsigned long long*>(reinterpret_cast<uint32_t*>(hdr) + kHdrSigWord);
}
// First thing in the kernel (after anything that must see the CTAs in their order of arrival).
// Returns false if the launch must end here.  Contains a block-wide barrier for CTA 0.
__device__ __forceinline__ bool clean_begin(const CleanArgs& c, WsHeader* hdr, uint32_t G, uint32_t b, int tid) {
    if (c.expect_clean != 0u && ld_cg(clean_mark_ptr(hdr)) != c.mark) {
        if (b == 0 && tid == 0) record_status(hdr, -1 /*GC_E_INVALID*/, 0xC1EA0000ull);
        return false;                // every CTA sees the same word
    }
    const uint32_t per = (c.ctrl_units + G - 1) / G;
    const uint32_t u0 = max(b * per, 16u), u1 = min(c.ctrl_units, (b + 1u) * per);     // (the header is 16 units)
    for (uint32_t u = u0 + (uint32_t)tid; u < u1; u += kBlock) {
        const bool is_early = (u >= c.early[0][0] && u < c.early[0][1]) || (u >= c.early[1][0] && u < c.early[1][1]) ||
                              (u >= c.early[2][0] && u < c.early[2][1]);
        if (!is_early) c.ctrl[u] = make_uint4(0u, 0u, 0u, 0u);
    }
    if (b == 0) {                    // the header: all but the barrier's, the exit counter's and the mark's words
        if (tid < 64 && tid != (int)kHdrBarrierWord && tid != (int)kHdrExitWord && tid != (int)kHdrSigWord &&
            tid != (int)kHdrSigWord + 1)
            reinterpret_cast<uint32_t*>(hdr)[tid] = 0u;
        __syncthreads();
    }
    return true;
}
// After the first barrier: every CTA has read the mark, the block is in use.
__device__ __forceinline__ void clean_in_use(WsHeader* hdr, uint32_t b, int tid) {
    if (b == 0 && tid == 0) *clean_mark_ptr(hdr) = 0ull;
}
// After the barrier that follows the last reader of the early sections.
__device__ __forceinline__ void clean_early(const CleanArgs& c, uint32_t G, uint32_t b, int tid) {
#pragma unroll
    for (int q = 0; q < 3; ++q) {
        const uint32_t len = c.early[q][1] - c.early[q][0], per = (len + G - 1) / G;
        for (uint32_t u = c.early[q][0] + b * per + (uint32_t)tid; u < min(c.early[q][1], c.early[q][0] + (b + 1u) * per); u += kBlock)
            c.ctrl[u] = make_uint4(0u, 0u, 0u, 0u);
    }
}
// Last step of a launch that ends normally (whole CTA calls; its writes come after every CTA's own
// cleaning: fence, then the counter).
__device__ __forceinline__ void leave_clean(const CleanArgs& c, WsHeader* hdr, uint32_t G, int tid) {
    if (tid == 0) {
        uint32_t* const w = reinterpret_cast<uint32_t*>(hdr);
        __threadfence();
        if (atomicAdd(w + kHdrExitWord, 1u) == G - 1u) {
            w[kHdrBarrierWord] = 0u; w[kHdrExitWord] = 0u;
            __threadfence();
            *clean_mark_ptr(hdr) = c.mark;
        }
    }
}

}  // namespace gc
