// libgc: host side of the C ABI declared in include/gc.h.
#include "gc.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <utility>
#include <vector>

#include "gc_single.cuh"
#include "gc_multi.cuh"
#include "gc_threshold.cuh"
#include "gc_thr_single.cuh"
#include "gc_thr_multi.cuh"
#include "gc_decode.cuh"

using namespace gc;

struct MultiGeom { uint32_t G = 0, per = 0, pool = 0, full = 0, ntab = 0; size_t smem = 0; };   // see multi_geometry

struct gc_plan_s {
    int device = 0;
    int mode = GC_TOPK;
    double density = 0.0;
    double cap_factor = 2.0;
    uint32_t stride = 64;
    uint32_t T = 0;
    uint64_t total_n = 0, total_cap = 0;
    uint32_t ntiles = 0;
    std::vector<TensorDesc> desc;
    TensorDesc* d_desc = nullptr;
    uint32_t* d_dectile = nullptr;          // plans of several tensors: tensor that holds the first element of each decode tile
    uint32_t* d_small = nullptr;            // ids of the small tensors (device), n_small entries
    std::vector<uint32_t> small_ids;
    uint32_t n_tiny = 0;                    // the first n_tiny of them are tiny (see tiny_tensor_warp)
    std::vector<uint32_t> reg_ids;          // tensors with elements that are not small (device copy follows the small ids)
    uint32_t nstiles = 0, ngroups = 0;
    uint32_t cand_cap = 0, cand_cap_alloc = 0;
    uint32_t skeys_tiles_alloc = 0;         // sample tiles the kept-keys section is sized for (fixed at plan creation)
    uint32_t n_sampled = 0;                 // tensors with a sample
    int path = 0;                           // GC_PATH_AUTO or GC_PATH_EXACT
    int decode_route = 0;                   // GC_DECODE_AUTO, GC_DECODE_NARROW or GC_DECODE_WIDE
    int decode_order = 0;                   // GC_ORDER_FIXED or GC_ORDER_ANY
    uint32_t rank_permille = 1000;          // scales the sample rank (testing aid)
    // workspace layout (byte offsets)
    size_t off_sel = 0, off_ssel = 0, off_gsel = 0, off_hist = 0, off_state = 0, off_gstate = 0,
           control_bytes = 0, off_tinfo = 0, off_cidx = 0, ws_bytes = 0;
    int sm_count = 0;
    int grid_thr = 0, grid_decode[2] = {0, 0};
    int grid_decode8 = 0, grid_decode8_apply = 0;      // k_decode_tiles with eight pre-loaded entries per thread (one tile buffer)
    int grid_decode_seg[2] = {0, 0}, grid_decode_seg_apply = 0;    // k_decode_segments: one / two tile buffers; with optimizer
    bool wide_ok = false;                         // k_decode_wide may use up to 64 KB of dynamic shared memory
    std::vector<std::pair<size_t, int>> wide_occ[2];      // (shared-memory bytes -> CTAs per SM), plain / with optimizer
    int grid_hist = 0, grid_compact = 0, grid_fold = 0, grid_sample = 0, grid_chist = 0, grid_ccompact = 0;
    int grid_fused = 0;                     // CTAs of the cooperative launch (0 = not available)
    // single-tensor shared-memory-pool kernel
    int grid_single_max = 0;                // resident CTAs (0 = not available)
    uint32_t single_grid = 0, single_maxt = 0, single_pool = 0;   // 0 = plan does not qualify
    RowMap single_rows = {};
    size_t single_smem = 0;
    size_t off_hist5 = 0, off_rowseg = 0, off_mid = 0, off_fine = 0, off_age = 0;
    uint32_t single_srank_hi = 0, single_srank_mid = 0;
    int grid_thr_single_max = 0;
    uint32_t thr_grid = 0, thr_maxt = 0, thr_pool = 0, thr_rounds = 0;    // one-tensor threshold kernel (0 = no)
    size_t thr_smem = 0;
    int grid_thr_multi_max = 0;
    uint32_t thrm_grid = 0, thrm_per = 0, thrm_pool = 0, thrm_ntab = 0;   // many-tensor threshold kernel (0 = no)
    size_t thrm_smem = 0;
    int grid_multi_max = 0;                 // resident CTAs of k_topk_multi (0 = not available)
    size_t multi_smem_max = 0, thrm_smem_max = 0;   // dynamic shared memory those occupancy figures were taken with
    bool ws_private = false;                // GC_OPT_WORKSPACE_PRIVATE
    std::vector<const void*> clean_ws;      // workspaces the one-tensor top-k kernel ran on last (and left clean), if private
    uint32_t wk_W = 0, wk_batch = 0;        // gc_compress_workers: workers per launch chosen for the last W seen
    MultiGeom wk_geom;
    uint32_t multi_ntab = 0;
    uint32_t multi_grid = 0, multi_per = 0, multi_pool = 0, multi_full = 0;       // 0 = plan does not qualify
    size_t multi_smem = 0;
    size_t off_shist = 0, off_bhist = 0, off_midn = 0, off_mmid = 0, off_skeys = 0;
    uint32_t n_empty = 0;                   // tensors without elements
    unsigned long long launches = 0;
    int last_cuda_error = 0;
    // optional per-kernel event timing
    // gc_compress_host: the host -> device copy runs on a stream of the plan's own, so that it
    // overlaps with the previous call's compress and device -> host copy
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_copied = nullptr;
    struct StagingUse { const void* ptr; cudaEvent_t done; };      // last compress that read a staging buffer
    std::vector<StagingUse> staging;
    struct Rec { cudaEvent_t a, b; int id; };
    std::vector<Rec> recs;
    size_t recs_used = 0;
};

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

constexpr size_t kSingleMidCap = 65536;      // short list of k_topk_single (candidates in the band bin of the threshold)
constexpr uint64_t kSampleMax = 131072;       // most sampled elements per tensor
constexpr uint64_t kSampleMaxSingle = 262144;   // ... when the plan holds one tensor (the sample is read in one step)
constexpr uint32_t kSinglePoolMax = 16384;   // most candidates one CTA of k_topk_single may hold
// Share of the oldest CTA of an SM above (and of the youngest below) the middle one's: measured
// best between 6 and 10 % on the 110M-element workload at 1 % density.  At 0.1 % density the
// fold loop has fewer candidates to handle, competes less for issue slots, and 4 % did better
// than 8 % (with 8 % the oldest CTAs of the 355M-element workload finished last).
constexpr double kSingleSkew = 0.08, kSingleSkewSparse = 0.04;
constexpr size_t kSingleRowBytes = (2 * kWarps + 3) * sizeof(uint32_t);   // shared memory per owned tile
constexpr uint32_t kMultiMaxTab = 1024;      // tensors whose tile tables k_topk_multi keeps in shared memory
constexpr size_t kMultiMaxPer = 160;         // most tiles one CTA of k_topk_multi may own
constexpr size_t kMultiRowBytes = (2 * kWarps + kSegWords) * sizeof(uint32_t);   // shared memory per owned tile
constexpr size_t kSingleMaxT = 341;          // most tiles one CTA of k_topk_single may own

inline uint64_t k_rule(uint64_t n, double density) {
    if (n == 0) return 0;
    double x = std::ceil(density * (double)n);
    uint64_t k = x < 1.0 ? 1ull : (uint64_t)x;
    return k < n ? k : n;
}

#define GC_CUDA(plan, expr)                                           \
    do {                                                              \
        cudaError_t e__ = (expr);                                     \
        if (e__ != cudaSuccess) {                                     \
            (plan)->last_cuda_error = (int)e__;                       \
            (void)cudaGetLastError();                                 \
            return GC_E_CUDA;                                         \
        }                                                             \
    } while (0)

// A plan's tables, grids and streams belong to one device: a compute call made while another
// device is current would launch there with this plan's device pointers.
inline bool on_plan_device(const gc_plan_s* p) {
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess) { (void)cudaGetLastError(); return false; }
    return cur == p->device;
}

// Brackets one enqueued operation with events when timing is on; always counts the launch.
struct Timed {
    gc_plan_s* p; cudaStream_t s; gc_plan_s::Rec* r = nullptr;
    Timed(gc_plan_s* p_, cudaStream_t s_, int id) : p(p_), s(s_) {
        ++p->launches;
        if (p->recs_used < p->recs.size()) {
            r = &p->recs[p->recs_used++];
            r->id = id;
            cudaEventRecord(r->a, s);
        }
    }
    ~Timed() { if (r) cudaEventRecord(r->b, s); }
};

WsView view(const gc_plan_s* p, void* ws) {
    char* b = static_cast<char*>(ws);
    WsView v;
    v.hdr = reinterpret_cast<WsHeader*>(b);
    v.sel = reinterpret_cast<TensorSel*>(b + p->off_sel);
    v.hist = reinterpret_cast<uint32_t*>(b + p->off_hist);
    v.tile_state = reinterpret_cast<unsigned long long*>(b + p->off_state);
    v.gate = nullptr;
    return v;
}

// Sampling parameters of the candidate path for one tensor (top-k mode).  The sample is one
// 4-element group out of `sstride`; tau_lo is the srank-th largest sampled key, where srank
// sits six standard deviations of the sampling noise above the expected rank density*m, so a
// candidate set smaller than k is a < 1e-8 event for well-mixed data (and only costs a redo).
void sample_params(TensorDesc& d, double density, uint32_t rank_permille, uint64_t* ccap, uint64_t target_max,
                   double coarse_factor, uint64_t* nsg_if_sampled) {
    const uint64_t n = d.n;
    d.sstride = 0; d.srank = 0;
    *ccap = n;
    *nsg_if_sampled = 0;
    if (d.ntiles <= 1) { d.kind = kKindSmall; *ccap = 0; return; }   // fits one tile: one CTA does the whole tensor
    uint64_t target = std::min<uint64_t>(target_max, std::max<uint64_t>(n / 128, std::min<uint64_t>(8192, n / 2)));
    uint64_t stride = std::max<uint64_t>(1, n / target);
    uint64_t groups = (n + 3) / 4;
    uint64_t nsg = (groups + stride - 1) / stride;
    *nsg_if_sampled = nsg;             // (whether it is sampled depends on the rank option; its sample size does not)
    double m = 4.0 * (double)nsg;
    double ks = density * m;
    double rank = std::ceil(ks + 6.0 * std::sqrt(ks) + 8.0) * (double)rank_permille / 1000.0;
    if (rank < 1.0) rank = 1.0;
    if (rank >= m) return;
    d.sstride = (uint32_t)stride;
    d.srank = (uint32_t)rank;
    double upper = (double)n * (rank + 6.0 * std::sqrt(rank)) / m;
    double cap = std::ceil(coarse_factor * 1.25 * upper) + 4096.0;
    *ccap = cap >= (double)n ? n : (uint64_t)cap;
}

// Fills the derived fields of the tensor table and the workspace layout.
void finish_layout(gc_plan_s* p) {
    uint64_t stile0 = 0, group0 = 0, ccap_total = 0, stiles_worst = 0;
    p->n_sampled = 0;
    p->small_ids.clear();
    p->reg_ids.clear();
    for (uint32_t t = 0; t < p->T; ++t) {
        TensorDesc& d = p->desc[t];
        d.kind = kKindRegular; d.pad = 0;
        uint64_t ccap = d.n;
        if (p->mode == GC_TOPK) {
            // (many tensors: the bracket is a histogram bin edge, up to twice the candidates)
            uint64_t nsg_w = 0;
            sample_params(d, p->density, p->rank_permille, &ccap, p->T == 1 ? kSampleMaxSingle : kSampleMax,
                          p->T == 1 ? 1.0 : 2.0, &nsg_w);
            stiles_worst += (nsg_w + (uint64_t)kSampleTile - 1) / (uint64_t)kSampleTile;
        } else {
            // threshold mode: the sample is part of the definition -- one 4-element group out of
            // `stride`, rank k_s = min(m, max(1, ceil(density * m))) over its m elements
            d.sstride = d.n ? d.stride : 0u;
            uint64_t groups = ((uint64_t)d.n + 3) / 4, m = 0;
            if (d.sstride) {
                uint64_t nsg = (groups + d.sstride - 1) / d.sstride;
                uint64_t last_first = (nsg - 1) * (uint64_t)d.sstride * 4;     // first element of the last sampled group
                m = (nsg - 1) * 4 + std::min<uint64_t>(4, d.n - last_first);
            }
            d.srank = (uint32_t)k_rule(m, p->density);
            if (d.n > 0 && d.ntiles == 1 && p->T >= 2) d.kind = kKindSmall;    // one CTA finishes it (many-tensor kernel)
        }
        uint64_t nst = 0;
        if (d.sstride) {
            uint64_t groups = ((uint64_t)d.n + 3) / 4;
            uint64_t nsg = (groups + d.sstride - 1) / d.sstride;
            nst = (nsg + (uint64_t)kSampleTile - 1) / (uint64_t)kSampleTile;
            ++p->n_sampled;
        }
        d.stile0 = (uint32_t)stile0; d.nstiles = (uint32_t)nst;
        d.group0 = (uint32_t)group0; d.ngroups = (d.ntiles + kWarps - 1) / kWarps;
        if (d.kind == kKindSmall && d.n > 0) p->small_ids.push_back(t);
        if (d.kind != kKindSmall && d.n > 0) p->reg_ids.push_back(t);
        stile0 += nst; group0 += d.ngroups; ccap_total += ccap;
    }
    p->nstiles = (uint32_t)stile0;
    p->ngroups = (uint32_t)group0;
    // tiny tensors (one warp each in the many-tensor top-k kernel) first in the list of small ones
    {
        auto tiny = [&](uint32_t t) { return p->mode == GC_TOPK && is_tiny(p->desc[t].n, p->desc[t].k); };
        std::stable_partition(p->small_ids.begin(), p->small_ids.end(), tiny);
        p->n_tiny = (uint32_t)std::count_if(p->small_ids.begin(), p->small_ids.end(), tiny);
    }
    // kept sample keys: room for every tensor that GC_OPT_SAMPLE_RANK_PERMILLE could turn into a
    // sampled one, fixed at plan creation so that the workspace never grows afterwards
    if (p->skeys_tiles_alloc == 0) p->skeys_tiles_alloc = (uint32_t)std::max<uint64_t>(stile0, stiles_worst);
    // every warp of the fold pass may strand part of a slab; CTAs never outnumber tiles
    ccap_total += (uint64_t)std::min<uint32_t>(p->ntiles, 1024u) * kWarps * kSlab;
    if (ccap_total > 0x7FFFFFFFull) ccap_total = 0x7FFFFFFFull;
    if (p->mode != GC_TOPK) {
        // one-tensor threshold plans keep a hit list: about k hits are expected (the sample says so),
        // up to the capacity factor are sent; the rest is slack for up to 1024 CTA regions
        ccap_total = 0;
        if (p->T >= 1 && p->total_cap > 0)
            ccap_total = std::min<uint64_t>(0x7FFFFFFFull, (uint64_t)(1.25 * (double)p->total_cap) + (1u << 20));
    }
    if (p->cand_cap_alloc == 0) p->cand_cap_alloc = (uint32_t)ccap_total;   // fixed at plan creation
    p->cand_cap = (uint32_t)std::min<uint64_t>(ccap_total, p->cand_cap_alloc);
    const size_t T = p->T;
    p->off_sel = sizeof(WsHeader);
    p->off_ssel = p->off_sel + sizeof(TensorSel) * T;
    p->off_gsel = p->off_ssel + sizeof(TensorSel) * T;
    p->off_hist = align_up(p->off_gsel + sizeof(TensorSel) * T, 256);
    p->off_state = align_up(p->off_hist + sizeof(uint32_t) * (size_t)kHistBins * T, 256);
    p->off_gstate = align_up(p->off_state + sizeof(unsigned long long) * (size_t)p->ntiles, 256);
    p->off_hist5 = align_up(p->off_gstate + sizeof(unsigned long long) * (size_t)p->ngroups, 256);
    // one-tensor kernels: six 2048-bin histogram slots, then 32-CTA segment totals
    p->off_rowseg = align_up(p->off_hist5 + (T == 1 ? sizeof(uint32_t) * 6 * (size_t)kHistBins : 0), 256);
    p->control_bytes = align_up(p->off_rowseg + (T == 1 ? sizeof(uint32_t) * kSingleMaxT * 20 : 0), 256);
    p->off_fine = p->control_bytes;
    p->control_bytes = align_up(p->off_fine + (T == 1 ? sizeof(uint32_t) * (size_t)kFineBins : 0), 256);
    p->off_age = p->control_bytes;                                   // CTAs arrived per SM (one-tensor kernels)
    p->control_bytes = align_up(p->off_age + (T == 1 ? sizeof(uint32_t) * 1024 : 0), 256);
    // many-tensor kernel: sample and band histogram per tensor, short-list lengths
    const size_t multi_hist = T >= 2 ? sizeof(uint32_t) * (size_t)kHistBins * T : 0;
    p->off_shist = p->control_bytes;
    p->off_bhist = align_up(p->off_shist + multi_hist, 256);
    p->off_midn = align_up(p->off_bhist + multi_hist, 256);
    p->control_bytes = align_up(p->off_midn + (multi_hist ? sizeof(uint32_t) * T : 0), 256);
    p->off_tinfo = p->control_bytes;
    p->off_cidx = align_up(p->off_tinfo + sizeof(uint2) * (size_t)p->ntiles * kWarps, 256);
    p->off_mid = align_up(p->off_cidx + sizeof(uint2) * (size_t)p->cand_cap_alloc, 256);
    p->off_mmid = align_up(p->off_mid + (T == 1 ? sizeof(uint2) * (size_t)kSingleMidCap : 0), 256);
    p->off_skeys = align_up(p->off_mmid + (multi_hist ? sizeof(uint2) * (size_t)kMultiMidCap * T : 0), 256);
    const bool keep_keys = multi_hist != 0 || (T == 1 && p->mode == GC_THRESHOLD);
    p->ws_bytes = align_up(p->off_skeys + (keep_keys ? sizeof(uint4) * (size_t)kBlock *
                                                       std::max(p->nstiles, p->skeys_tiles_alloc) : 0), 256);
}


// Shares of a one-tensor plan's CTAs: equal, or - when the launch fills every SM three CTAs deep
// and every column has at least twelve rows - in the proportion in which the oldest, middle and
// youngest CTA of an SM advance.  `maxt` comes in as the rows of an equal share and goes out as
// the rows of the largest one.
static RowMap make_row_map(const gc_plan_s* p, uint32_t ntiles, uint32_t G, uint32_t& maxt, double skew) {
    RowMap rm;
    rm.G = G; rm.gA = G; rm.n0 = rm.n1 = rm.n2 = maxt; rm.s1 = rm.s2 = maxt * G;
    if (skew > 0.0 && G == 3u * (uint32_t)p->sm_count && ntiles >= 12u * G) {
        const uint32_t gA = (uint32_t)p->sm_count;
        const uint32_t total = (ntiles + gA - 1) / gA;               // rows of the three classes together
        const uint32_t n1 = maxt;
        const uint32_t dd = std::max<uint32_t>(1u, (uint32_t)((double)ntiles / G * skew + 0.5));
        const uint32_t n0 = n1 + dd;
        if (total > n0 + n1 && total - n0 - n1 <= n1) {
            rm.gA = gA; rm.n0 = n0; rm.n1 = n1; rm.n2 = total - n0 - n1;
            rm.s1 = rm.n2 * G; rm.s2 = rm.s1 + (rm.n1 - rm.n2) * 2u * gA;
            maxt = n0;
        }
    }
    rm.mG = (uint32_t)((1ull << 32) / rm.G) + 1u;
    rm.m2A = (uint32_t)((1ull << 32) / (2u * rm.gA)) + 1u;
    rm.mA = (uint32_t)((1ull << 32) / rm.gA) + 1u;
    return rm;
}

// Decides whether the plan can use the single-tensor kernel and with which geometry.
void plan_single(gc_plan_s* p) {
    p->single_grid = 0;
    if (p->mode != GC_TOPK || p->T != 1 || p->grid_single_max <= 0) return;
    const TensorDesc& d = p->desc[0];
    if (d.sstride == 0 || d.ntiles == 0 || d.off != 0) return;
    uint32_t G = std::min<uint32_t>((uint32_t)p->grid_single_max, d.ntiles);
    // Small tensors are all latency (a CTA has a handful of tiles and five phases to walk through):
    // there two CTAs per SM get through the phases sooner than three (2M-10M elements: 31-49 us
    // against 37-51 us).  From about 12M elements on the third CTA pays for itself; below 300
    // tiles there is a CTA per tile anyway (fewer were no faster).
    if (d.ntiles <= 3000u) G = std::min<uint32_t>(G, 2u * (uint32_t)p->sm_count);
    uint32_t maxt = (d.ntiles + G - 1) / G;
    const RowMap rm = make_row_map(p, d.ntiles, G, maxt, p->density >= 0.005 ? kSingleSkew : kSingleSkewSparse);
    if (maxt > kSingleMaxT || G > 640) return;                       // chunk records and totals must stay small
    if (d.ntiles >= (1u << 20)) return;                              // (the row arithmetic divides by multiplication)
    // region per CTA; one bit per slot has to fit in shared memory beside the chunk records
    const uint32_t pool = std::min<uint32_t>(p->cand_cap_alloc / G, kSinglePoolMax);
    const size_t rec_bytes = (size_t)maxt * kSingleRowBytes + sizeof(uint32_t) * ((pool + 31) / 32);
    // expected candidates per CTA (sample rank over sample size, times n), with head-room
    const uint64_t groups = ((uint64_t)d.n + 3) / 4, nsg = (groups + d.sstride - 1) / d.sstride;
    if (nsg > (uint64_t)2 * G * kBlock) return;                     // a thread owns at most two sample groups
    const double expect = (double)d.n * (double)d.srank / (4.0 * (double)nsg) / (double)G;
    if ((double)pool < 1.5 * expect + 512.0) return;
    // upper bracket: the sample rank that stays below the expected one by the same margin
    const double ks = p->density * 4.0 * (double)nsg;
    const double hi = std::floor(ks - 6.0 * std::sqrt(ks) - 8.0);
    p->single_srank_hi = hi >= 1.0 ? (uint32_t)hi : 1u;    // small sample: the largest sampled key bounds the band
    p->single_srank_mid = (uint32_t)std::max(1.0, std::ceil(ks));
    p->single_grid = G; p->single_maxt = maxt; p->single_pool = pool; p->single_smem = rec_bytes;
    p->single_rows = rm;
}

// Decides whether a threshold plan can use the one-tensor kernel and with which geometry.
void plan_thr_single(gc_plan_s* p) {
    p->thr_grid = 0;
    if (p->mode != GC_THRESHOLD || p->T != 1 || p->grid_thr_single_max <= 0) return;
    const TensorDesc& d = p->desc[0];
    if (d.sstride == 0 || d.ntiles == 0 || d.off != 0) return;
    uint32_t G = std::min<uint32_t>((uint32_t)p->grid_thr_single_max, d.ntiles);
    if (d.ntiles <= 2500u) G = std::min<uint32_t>(G, 2u * (uint32_t)p->sm_count);    // small tensors: as in plan_single (2M: 28.9 against 33.1 us)
    const uint32_t maxt = (d.ntiles + G - 1) / G;     // equal shares (unequal ones as in the top-k kernel: 268.5 us
                                                      // against 262.5 us on the 110M-element workload)
    if (maxt > kSingleMaxT || G > 640) return;
    const uint32_t pool = std::min<uint32_t>(p->cand_cap_alloc / G, kSinglePoolMax);
    if ((double)pool < 1.25 * (double)d.k / (double)G + 256.0) return;
    const uint64_t groups = ((uint64_t)d.n + 3) / 4, nsg = (groups + d.sstride - 1) / d.sstride;
    const uint64_t rounds = (nsg + (uint64_t)G * kBlock - 1) / ((uint64_t)G * kBlock);
    if (rounds > 64) return;
    p->thr_grid = G; p->thr_maxt = maxt; p->thr_pool = pool; p->thr_rounds = (uint32_t)rounds;
    p->thr_smem = (size_t)maxt * (2 * kWarps + 2) * sizeof(uint32_t);
}

// Geometry of the many-tensor threshold kernel when G CTAs share one worker's tiles (G = 0: no).
MultiGeom thr_multi_geometry(const gc_plan_s* p, uint32_t G) {
    MultiGeom mg;
    if (p->mode != GC_THRESHOLD || p->T < 2 || G == 0 || p->ntiles == 0) return mg;
    G = std::min<uint32_t>(G, p->ntiles);
    const uint32_t per = (p->ntiles + G - 1) / G;
    if (per > kMultiMaxPer) return mg;
    // one CTA ranks a whole tensor's kept sample keys: keep that bounded
    for (uint32_t t : p->reg_ids)
        if (p->desc[t].nstiles > 128 || p->desc[t].sstride == 0) return mg;
    const uint32_t pool = std::min<uint32_t>(p->cand_cap_alloc / G, kSinglePoolMax);
    // expected hits of the busiest CTA: about k per tensor, spread over its tiles
    double worst = 0.0;
    uint32_t t = 0;
    for (uint32_t b = 0; b < G; ++b) {
        double e = 0.0;
        for (uint32_t tile = b * per; tile < std::min<uint32_t>(p->ntiles, (b + 1) * per); ++tile) {
            while (t + 1 < p->T && (p->desc[t].ntiles == 0 || tile >= p->desc[t].tile0 + p->desc[t].ntiles)) ++t;
            const TensorDesc& d = p->desc[t];
            if (d.kind != kKindSmall && d.ntiles) e += std::min<double>(kTile, (double)d.k / (double)d.ntiles);
        }
        worst = std::max(worst, e);
    }
    if ((double)pool < 2.0 * worst + 512.0) return mg;
    mg.G = G; mg.per = per; mg.pool = pool; mg.full = G;
    mg.ntab = p->T <= kMultiMaxTab ? p->T : 0u;
    mg.smem = (size_t)per * kMultiRowBytes + 2 * sizeof(uint32_t) * (size_t)mg.ntab;
    return mg;
}

// Decides whether a threshold plan can use the many-tensor kernel and with which geometry.
void plan_thr_multi(gc_plan_s* p) {
    p->thrm_grid = 0;
    if (p->grid_thr_multi_max <= 0) return;
    const MultiGeom mg = thr_multi_geometry(p, (uint32_t)p->grid_thr_multi_max);
    if (mg.G == 0) return;
    p->thrm_grid = mg.G; p->thrm_per = mg.per; p->thrm_pool = mg.pool; p->thrm_ntab = mg.ntab; p->thrm_smem = mg.smem;
}

// Geometry of the many-tensor kernel when G CTAs share one worker's tiles: MultiGeom.

// Decides whether G CTAs can run the many-tensor kernel on this plan (G = 0 in the result: no).
// `age_skew`: the CTA index follows the CTAs' age on their SMs (a launch that fills the device
// with this plan alone), so the leftover tiles go to the youngest third.
MultiGeom multi_geometry(const gc_plan_s* p, uint32_t G, bool age_skew) {
    MultiGeom mg;
    if (p->mode != GC_TOPK || p->T < 2 || G == 0 || p->ntiles == 0) return mg;
    G = std::min<uint32_t>(G, p->ntiles);
    const uint32_t per = (p->ntiles + G - 1) / G;
    if (per > kMultiMaxPer) return mg;
    const uint32_t pool = std::min<uint32_t>(p->cand_cap_alloc / G, kSinglePoolMax);
    // expected candidates of the busiest CTA (bracket rank over sample size, times two for the
    // bin edge), with head-room
    std::vector<double> per_tile(p->T, 0.0);
    for (uint32_t t = 0; t < p->T; ++t) {
        const TensorDesc& d = p->desc[t];
        if (d.kind == kKindSmall || d.ntiles == 0) continue;
        if (d.sstride == 0) { per_tile[t] = (double)kTile; continue; }
        const uint64_t groups = ((uint64_t)d.n + 3) / 4, nsg = (groups + d.sstride - 1) / d.sstride;
        per_tile[t] = std::min<double>(kTile, 2.0 * (double)kTile * (double)d.srank / (4.0 * (double)nsg));
    }
    // runs: `per` tiles for the first two thirds of a full grid, the rest spread over the last third
    // (the youngest CTAs of their SMs, which advance the slowest); every CTA `per` tiles otherwise
    uint32_t full_ctas = G;
    if (age_skew && per >= 8) {
        const uint32_t fc = (uint32_t)((uint64_t)G * 2u / 3u);
        if ((uint64_t)fc * per < p->ntiles) full_ctas = fc;
    }
    auto run_of = [&](uint32_t b, uint32_t& f, uint32_t& l) {
        if (b < full_ctas) { f = std::min<uint32_t>(p->ntiles, b * per); l = std::min<uint32_t>(p->ntiles, f + per); return; }
        const uint32_t s0 = std::min<uint32_t>(p->ntiles, full_ctas * per), rest = p->ntiles - s0, nb = G - full_ctas;
        f = s0 + (uint32_t)(((uint64_t)(b - full_ctas) * rest) / nb);
        l = s0 + (uint32_t)(((uint64_t)(b - full_ctas + 1) * rest) / nb);
    };
    double worst = 0.0;
    uint32_t t = 0;
    for (uint32_t b = 0; b < G; ++b) {
        double e = 0.0;
        uint32_t f, l;
        run_of(b, f, l);
        if (l - f > per) return mg;
        for (uint32_t tile = f; tile < l; ++tile) {
            while (t + 1 < p->T && (p->desc[t].ntiles == 0 || tile >= p->desc[t].tile0 + p->desc[t].ntiles)) ++t;
            e += per_tile[t];
        }
        worst = std::max(worst, e);
    }
    if ((double)pool < 1.5 * worst + 512.0) return mg;
    mg.G = G; mg.per = per; mg.pool = pool; mg.full = full_ctas;
    mg.ntab = p->T <= kMultiMaxTab ? p->T : 0u;
    mg.smem = (size_t)per * kMultiRowBytes + sizeof(uint32_t) * ((pool + 31) / 32) + 2 * sizeof(uint32_t) * (size_t)mg.ntab;
    return mg;
}

// Decides whether the plan can use the many-tensor kernel and with which geometry.
void plan_multi(gc_plan_s* p) {
    p->multi_grid = 0;
    if (p->grid_multi_max <= 0) return;
    const MultiGeom mg = multi_geometry(p, (uint32_t)p->grid_multi_max, p->ntiles >= (uint32_t)p->grid_multi_max);
    if (mg.G == 0) return;
    p->multi_grid = mg.G; p->multi_per = mg.per; p->multi_pool = mg.pool; p->multi_full = mg.full;
    p->multi_ntab = mg.ntab; p->multi_smem = mg.smem;
}

int upload_table(gc_plan_s* p) {
    if (p->device < 0 || p->T == 0) return GC_OK;
    cudaError_t e = cudaMemcpy(p->d_desc, p->desc.data(), sizeof(TensorDesc) * (size_t)p->T,
                               cudaMemcpyHostToDevice);
    if (e == cudaSuccess && !p->small_ids.empty())
        e = cudaMemcpy(p->d_small, p->small_ids.data(), sizeof(uint32_t) * p->small_ids.size(),
                       cudaMemcpyHostToDevice);
    if (e == cudaSuccess && !p->reg_ids.empty())
        e = cudaMemcpy(p->d_small + p->T, p->reg_ids.data(), sizeof(uint32_t) * p->reg_ids.size(),
                       cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { p->last_cuda_error = (int)e; (void)cudaGetLastError(); return GC_E_CUDA; }
    return GC_OK;
}

template <typename K>
int blocks_per_sm(K kernel, int threads) {
    int nb = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kernel, threads, 0) != cudaSuccess || nb < 1) {
        (void)cudaGetLastError();
        nb = 1;
    }
    return nb;
}

}  // namespace

// Which decode kernel a call takes.  The narrow kernel pre-loads 4 x (256 / W) entries per worker
// and tile in registers; lists that are expected to hold more per tile than that (many workers,
// or dense lists) go to the wide kernel, which keeps `win` entries per worker in shared memory.
struct DecodeRoute {
    bool wide = false;
    bool any = false;           // (with wide) the kernel that adds without a fixed worker order
    uint32_t win = 0;
    size_t smem = 0;
    int grid = 0;
    int rounds = kDecRounds;    // (narrow) entries a thread pre-loads per tile: kDecRounds or twice that
};
template <bool APPLY>
static DecodeRoute decode_route(gc_plan_t* p, uint32_t W, bool zero_first) {
    DecodeRoute r;
    if (W == 0 || p->total_n == 0) return r;
    const uint64_t avg = (p->total_cap * (uint64_t)kDecTile + p->total_n - 1) / p->total_n;     // per worker and tile
    const uint64_t need = avg + avg / 2 + 16;
    uint32_t Wp = 1;
    while (Wp < W && Wp < 64) Wp <<= 1;
    uint64_t narrow_window = (uint64_t)kDecRounds * (kDecBlock / Wp);
    r.any = p->decode_order == GC_ORDER_ANY;
    // Tiles that start at +0 take the narrow kernel's counted route from a few workers on; there a
    // window of twice the size (eight pre-loaded entries per thread) still beats the rings, so
    // lists up to that density stay with the narrow kernel (16 workers at 1 %: measured below).
    if (!r.any && zero_first && W >= kDecCountedFrom && avg + avg / 4 > narrow_window &&
        avg + avg / 4 <= 2 * narrow_window && p->grid_decode8 > 0) {
        r.rounds = 2 * kDecRounds;
        narrow_window *= 2;
    }
    // measured: the narrow kernel wins as long as most tiles fit its window
    r.wide = r.any || (p->decode_route == GC_DECODE_AUTO ? avg + avg / 4 > narrow_window
                                                          : p->decode_route == GC_DECODE_WIDE);
    if (!p->wide_ok) r.wide = false;
    if (!r.wide) return r;
    uint32_t win = 32;
    while (win < need && win < 1024) win <<= 1;
    while ((uint64_t)W * win > kDecWideEntries && win > 32) win >>= 1;
    r.win = win;
    r.smem = kDecTileBytes + 8 * (size_t)W * win;
    int nb = -1;
    const size_t key = r.smem + (r.any ? 1 : 0);          // (shared-memory sizes are multiples of 256)
    for (auto& e : p->wide_occ[APPLY ? 1 : 0]) if (e.first == key) nb = e.second;
    if (nb < 0) {
        const cudaError_t eo = r.any
            ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_decode_any<APPLY>, kDecBlock, r.smem)
            : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_decode_wide<APPLY>, kDecBlock, r.smem);
        if (eo != cudaSuccess) {
            (void)cudaGetLastError();
            nb = 0;
        }
        p->wide_occ[APPLY ? 1 : 0].emplace_back(key, nb);
    }
    r.grid = p->sm_count * nb;
    if (r.grid <= 0) r.wide = false;
    return r;
}

extern "C" {

static int compress_route(const gc_plan_s* p);

uint32_t gc_version(void) { return 1u; }

int gc_plan(gc_plan_t** out, int device, uint32_t n_tensors, const uint64_t* sizes,
            double density, int mode, uint32_t sample_stride, double cap_factor) {
    if (out == nullptr) return GC_E_INVALID;
    *out = nullptr;
    if (n_tensors > 0 && sizes == nullptr) return GC_E_INVALID;
    if (!(density > 0.0) || !(density <= 1.0)) return GC_E_INVALID;
    if (mode != GC_TOPK && mode != GC_THRESHOLD) return GC_E_INVALID;
    if (cap_factor == 0.0) cap_factor = 2.0;
    if (!(cap_factor >= 1.0)) return GC_E_INVALID;
    if (sample_stride == 0) sample_stride = 64;
    uint64_t total = 0;
    for (uint32_t t = 0; t < n_tensors; ++t) {
        total += sizes[t];
        if (total > 0x7FFFFFFFull) return GC_E_TOO_LARGE;
    }
    gc_plan_s* p = new (std::nothrow) gc_plan_s();
    if (p == nullptr) return GC_E_INVALID;
    p->device = device; p->mode = mode; p->density = density;
    p->cap_factor = cap_factor; p->stride = sample_stride; p->T = n_tensors;
    p->total_n = total;
    p->desc.resize(n_tensors);
    uint64_t off = 0, out_off = 0, tile0 = 0;
    for (uint32_t t = 0; t < n_tensors; ++t) {
        TensorDesc& d = p->desc[t];
        uint64_t n = sizes[t];
        if (n == 0) ++p->n_empty;
        uint64_t k = k_rule(n, density);
        uint64_t cap = k;
        if (mode == GC_THRESHOLD) {
            double c = std::ceil(cap_factor * (double)k);
            cap = c >= (double)n ? n : (uint64_t)c;
        }
        uint64_t lead = off & 3ull;                       // elements before the tensor in its first group
        uint64_t nt = n == 0 ? 0 : (lead + n + kTile - 1) / kTile;
        d.off = (uint32_t)off; d.n = (uint32_t)n; d.k = (uint32_t)k; d.cap = (uint32_t)cap;
        d.out_off = (uint32_t)out_off; d.tile0 = (uint32_t)tile0; d.ntiles = (uint32_t)nt;
        d.stride = n <= 65536 ? 1u : sample_stride;
        d.kind = kKindRegular; d.pad = 0;
        off += n; out_off += cap; tile0 += nt;
    }
    p->total_cap = out_off;
    p->ntiles = (uint32_t)tile0;
    finish_layout(p);

    if (device < 0) {            // host-only plan: answers queries, refuses compute calls
        *out = p;
        return GC_OK;
    }
    int caller_device = -1;
    if (cudaGetDevice(&caller_device) != cudaSuccess) { (void)cudaGetLastError(); caller_device = -1; }
    struct RestoreDevice {           // the caller's current device is left as it was found
        int dev;
        ~RestoreDevice() { if (dev >= 0) (void)cudaSetDevice(dev); }
    } restore_device{caller_device};
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess && n_tensors > 0) {
        e = cudaMalloc(reinterpret_cast<void**>(&p->d_desc), sizeof(TensorDesc) * (size_t)n_tensors);
        if (e == cudaSuccess)
            e = cudaMalloc(reinterpret_cast<void**>(&p->d_small), sizeof(uint32_t) * 2 * (size_t)n_tensors);
        if (e == cudaSuccess) e = upload_table(p) == GC_OK ? cudaSuccess : cudaErrorUnknown;
        if (e == cudaSuccess && n_tensors > 1 && p->total_n > 0) {
            const uint32_t ntl = (uint32_t)((p->total_n + kDecTile - 1) / kDecTile);
            std::vector<uint32_t> tt(ntl);
            uint32_t t = 0;
            for (uint32_t tl = 0; tl < ntl; ++tl) {
                const uint64_t e0 = (uint64_t)tl * kDecTile;
                while (t + 1 < n_tensors && (p->desc[t].n == 0 || e0 >= (uint64_t)p->desc[t].off + p->desc[t].n)) ++t;
                tt[tl] = t;
            }
            e = cudaMalloc(reinterpret_cast<void**>(&p->d_dectile), sizeof(uint32_t) * (size_t)ntl);
            if (e == cudaSuccess)
                e = cudaMemcpy(p->d_dectile, tt.data(), sizeof(uint32_t) * (size_t)ntl, cudaMemcpyHostToDevice);
        }
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        if (p->d_desc) cudaFree(p->d_desc);
        if (p->d_small) cudaFree(p->d_small);
        if (p->d_dectile) cudaFree(p->d_dectile);
        delete p;
        return GC_E_CUDA;
    }
    p->grid_hist = p->sm_count * blocks_per_sm(k_hist<0, SRC_FOLD>, kBlock);
    p->grid_compact = p->sm_count * blocks_per_sm(k_compact, kBlock);
    p->grid_fold = p->sm_count * blocks_per_sm(k_fold_cand, kBlock);
    {
        int coop = 0;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, device) != cudaSuccess) {
            (void)cudaGetLastError();
            coop = 0;
        }
        p->grid_fused = coop ? p->sm_count * blocks_per_sm(k_compress_fused, kBlock) : 0;
        p->grid_single_max = 0;
        if (coop) {
            int nb = 0;       // sized for the largest chunk-record block the kernel may be given
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_topk_single<GradF32>, kBlock, kSingleMaxT * kSingleRowBytes + kSinglePoolMax / 8) ==
                    cudaSuccess && nb >= 1)
                p->grid_single_max = p->sm_count * nb;
        }
        (void)cudaGetLastError();
        plan_single(p);
        p->grid_thr_single_max = 0;
        if (coop) {
            int nb = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_threshold_single, kBlock,
                                                              kSingleMaxT * (2 * kWarps + 2) * sizeof(uint32_t)) ==
                    cudaSuccess && nb >= 1)
                p->grid_thr_single_max = p->sm_count * nb;
            else
                (void)cudaGetLastError();
        }
        plan_thr_single(p);
        p->grid_thr_multi_max = 0;
        if (coop) {
            int nb = 0;
            p->thrm_smem_max = kMultiMaxPer * kMultiRowBytes + 8 * kMultiMaxTab;
            int nbw = 0;          // (the several-workers form of the kernel must be as resident as the kernel itself)
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_threshold_multi, kBlock, p->thrm_smem_max) ==
                    cudaSuccess && nb >= 1 &&
                cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nbw, k_threshold_workers, kBlock, p->thrm_smem_max) ==
                    cudaSuccess && nbw >= 1)
                p->grid_thr_multi_max = p->sm_count * std::min(nb, nbw);
            else
                (void)cudaGetLastError();
        }
        plan_thr_multi(p);
        p->grid_multi_max = 0;
        if (coop) {
            int nb = 0;
            p->multi_smem_max = kMultiMaxPer * kMultiRowBytes + kSinglePoolMax / 8 + 8 * kMultiMaxTab;
            int nbw = 0;          // (the several-workers form of the kernel must be as resident as the kernel itself)
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_topk_multi<GradF32>, kBlock, p->multi_smem_max) ==
                    cudaSuccess && nb >= 1 &&
                cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nbw, k_topk_workers<GradF32>, kBlock, p->multi_smem_max) ==
                    cudaSuccess && nbw >= 1)
                p->grid_multi_max = p->sm_count * std::min(nb, nbw);
            else
                (void)cudaGetLastError();
        }
        plan_multi(p);
    }
    p->grid_thr = p->sm_count * blocks_per_sm(k_threshold_emit, kBlock);
    {
        cudaError_t ed = cudaFuncSetAttribute(k_decode_tiles<false, kDecRounds>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)(2 * kDecTileBytes));
        for (int nbuf = 1; nbuf <= 2; ++nbuf) {
            int nb = 0;
            if (ed == cudaSuccess)
                ed = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_decode_tiles<false, kDecRounds>, kDecBlock,
                                                                   nbuf * kDecTileBytes);
            if (ed != cudaSuccess || nb < 1) { (void)cudaGetLastError(); nb = 0; }
            p->grid_decode[nbuf - 1] = p->sm_count * nb;     // 0: fall back to one launch per worker
        }
        int nb8 = 0, nb8a = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb8, k_decode_tiles<false, 2 * kDecRounds>, kDecBlock,
                                                          kDecTileBytes) != cudaSuccess || nb8 < 1) { (void)cudaGetLastError(); nb8 = 0; }
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb8a, k_decode_tiles<true, 2 * kDecRounds>, kDecBlock,
                                                          kDecTileBytes) != cudaSuccess || nb8a < 1) { (void)cudaGetLastError(); nb8a = 0; }
        p->grid_decode8 = p->sm_count * nb8;
        p->grid_decode8_apply = p->sm_count * nb8a;
    }
    {
        // lists with per-tensor counts (plans of several tensors): the segment-walking tile kernel
        cudaError_t ed = cudaFuncSetAttribute(k_decode_segments<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)(2 * kDecTileBytes));
        for (int nbuf = 1; nbuf <= 2; ++nbuf) {
            int nb = 0;
            if (ed == cudaSuccess)
                ed = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_decode_segments<false>, kDecBlock,
                                                                   nbuf * kDecTileBytes);
            if (ed != cudaSuccess || nb < 1) { (void)cudaGetLastError(); nb = 0; }
            p->grid_decode_seg[nbuf - 1] = p->sm_count * nb;
        }
        int nb = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_decode_segments<true>, kDecBlock, kDecTileBytes) !=
                cudaSuccess || nb < 1) { (void)cudaGetLastError(); nb = 0; }
        p->grid_decode_seg_apply = p->sm_count * nb;
    }
    p->wide_ok = cudaFuncSetAttribute(k_decode_wide<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)(kDecTileBytes + 8 * kDecWideEntries)) == cudaSuccess &&
                 cudaFuncSetAttribute(k_decode_wide<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)(kDecTileBytes + 8 * kDecWideEntries)) == cudaSuccess &&
                 cudaFuncSetAttribute(k_decode_any<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)(kDecTileBytes + 8 * kDecWideEntries)) == cudaSuccess &&
                 cudaFuncSetAttribute(k_decode_any<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)(kDecTileBytes + 8 * kDecWideEntries)) == cudaSuccess;
    (void)cudaGetLastError();
    p->grid_sample = p->sm_count * blocks_per_sm(k_hist<0, SRC_SAMPLE>, kBlock);
    p->grid_chist = p->sm_count * blocks_per_sm(k_cand_hist<1>, kBlock);
    p->grid_ccompact = p->sm_count * blocks_per_sm(k_cand_compact<true>, kBlock);
    *out = p;
    return GC_OK;
}

int gc_plan_set_option(gc_plan_t* p, int option, uint64_t value) {
    if (p == nullptr) return GC_E_INVALID;
    switch (option) {
        case GC_OPT_PATH:
            if (value != GC_PATH_AUTO && value != GC_PATH_EXACT && value != GC_PATH_STAGED) return GC_E_INVALID;
            p->path = (int)value;
            p->clean_ws.clear();
            return GC_OK;
        case GC_OPT_SAMPLE_RANK_PERMILLE:
            if (value < 1 || value > 100000) return GC_E_INVALID;
            if (p->device >= 0 && !on_plan_device(p)) return GC_E_INVALID;      // (the table is uploaded again)
            p->rank_permille = (uint32_t)value;
            p->wk_W = 0;
            finish_layout(p);                          // workspace size stays as planned (see skeys_tiles_alloc)
            plan_single(p);
            plan_multi(p);
            return upload_table(p);
        case GC_OPT_CANDIDATE_CAPACITY:
            if (value > p->cand_cap_alloc) return GC_E_INVALID;
            p->cand_cap = (uint32_t)value;
            p->wk_W = 0;
            return GC_OK;
        case GC_OPT_WORKSPACE_PRIVATE:
            if (value > 1) return GC_E_INVALID;
            p->ws_private = value != 0;
            p->clean_ws.clear();
            return GC_OK;
        case GC_OPT_DECODE_ORDER:
            if (value != GC_ORDER_FIXED && value != GC_ORDER_ANY) return GC_E_INVALID;
            p->decode_order = (int)value;
            return GC_OK;
        case GC_OPT_DECODE_ROUTE:
            if (value != GC_DECODE_AUTO && value != GC_DECODE_NARROW && value != GC_DECODE_WIDE) return GC_E_INVALID;
            p->decode_route = (int)value;
            return GC_OK;
        default:
            return GC_E_INVALID;
    }
}

int gc_plan_query(const gc_plan_t* p, int what, uint32_t tensor, uint64_t* value) {
    if (p == nullptr || value == nullptr) return GC_E_INVALID;
    switch (what) {
        case GC_Q_N_TENSORS: *value = p->T; return GC_OK;
        case GC_Q_TOTAL_N: *value = p->total_n; return GC_OK;
        case GC_Q_TOTAL_CAP: *value = p->total_cap; return GC_OK;
        case GC_Q_WORKSPACE_BYTES: *value = p->ws_bytes; return GC_OK;
        case GC_Q_MODE: *value = (uint64_t)p->mode; return GC_OK;
        case GC_Q_KERNEL_LAUNCHES: *value = p->launches; return GC_OK;
        case GC_Q_CANDIDATE_CAPACITY: *value = p->cand_cap; return GC_OK;
        case GC_Q_COMPRESS_ROUTE: *value = (uint64_t)compress_route(p); return GC_OK;
        default: break;
    }
    if (tensor >= p->T) return GC_E_INVALID;
    const TensorDesc& d = p->desc[tensor];
    switch (what) {
        case GC_Q_TENSOR_N: *value = d.n; return GC_OK;
        case GC_Q_TENSOR_K: *value = d.k; return GC_OK;
        case GC_Q_TENSOR_CAP: *value = d.cap; return GC_OK;
        case GC_Q_TENSOR_OFFSET: *value = d.off; return GC_OK;
        case GC_Q_TENSOR_OUT_OFFSET: *value = d.out_off; return GC_OK;
        case GC_Q_TENSOR_STRIDE: *value = d.stride; return GC_OK;
        default: return GC_E_INVALID;
    }
}

// The control block as the self-cleaning kernels see it (see CleanArgs): up to three early sections.
static CleanArgs clean_args(const gc_plan_s* p, void* workspace, int route, bool expect_clean) {
    CleanArgs c{};
    c.ctrl = reinterpret_cast<uint4*>(workspace);
    c.ctrl_units = (uint32_t)(p->control_bytes / 16);
    auto range = [&](int q, size_t off, size_t bytes) { c.early[q][0] = (uint32_t)(off / 16); c.early[q][1] = (uint32_t)((off + bytes) / 16); };
    if (route == GC_ROUTE_TOPK_ONE) {
        range(0, p->off_hist5, sizeof(uint32_t) * kHistBins);                 // coarse sample histogram
        range(1, p->off_fine, sizeof(uint32_t) * (size_t)kFineBins);          // fine sample histogram
        range(2, p->off_age, sizeof(uint32_t) * 1024);                        // arrivals per SM
    } else {
        range(0, p->off_shist, sizeof(uint32_t) * (size_t)kHistBins * p->T);  // coarse sample histogram per tensor
    }
    c.mark = 0xC1EA9B10C5ull ^ ((unsigned long long)p->control_bytes << 24) ^ ((unsigned long long)route << 56) ^
             (unsigned long long)p->total_n;
    c.expect_clean = expect_clean ? 1u : 0u;
    return c;
}

// Workspaces this plan's self-cleaning kernels ran on last (GC_OPT_WORKSPACE_PRIVATE).
static bool take_clean(gc_plan_s* p, const void* workspace) {       // forgets it: the coming launch dirties it
    const auto known = std::find(p->clean_ws.begin(), p->clean_ws.end(), workspace);
    if (known == p->clean_ws.end()) return false;
    p->clean_ws.erase(known);
    return true;
}
static void note_clean(gc_plan_s* p, const void* workspace) {
    if (!p->ws_private) return;
    if (p->clean_ws.size() >= 2 * GC_MAX_WORKERS) p->clean_ws.erase(p->clean_ws.begin());     // (oldest forgotten)
    p->clean_ws.push_back(workspace);
}

// Which kernels a gc_compress call on this plan takes (GC_ROUTE_*); the dispatch below and
// GC_Q_COMPRESS_ROUTE both ask here.
static int compress_route(const gc_plan_s* p) {
    if (p->device < 0 || p->total_n == 0) return GC_ROUTE_NONE;
    if (p->mode == GC_THRESHOLD) {
        if (p->path == GC_PATH_AUTO && p->thr_grid > 0) return GC_ROUTE_THRESHOLD_ONE;
        if (p->path == GC_PATH_AUTO && p->thrm_grid > 0) return GC_ROUTE_THRESHOLD_MANY;
        return GC_ROUTE_THRESHOLD_STAGED;
    }
    if (p->path == GC_PATH_EXACT) return GC_ROUTE_EXACT;
    if (p->path == GC_PATH_AUTO && p->single_grid > 0) return GC_ROUTE_TOPK_ONE;
    if (p->path == GC_PATH_AUTO && p->multi_grid > 0) return GC_ROUTE_TOPK_MANY;
    if (p->path == GC_PATH_AUTO && p->grid_fused > 0) return GC_ROUTE_TOPK_GENERAL;
    return GC_ROUTE_TOPK_STAGED;
}

// Argument block of the many-tensor kernel for one worker's buffers and a given geometry.
static MultiArgs multi_args(const gc_plan_s* p, const MultiGeom& mg, const void* grad, float* residual,
                            uint32_t* out_idx, float* out_val, uint32_t* out_count, void* workspace, bool expect_clean) {
    char* wb = static_cast<char*>(workspace);
    WsView ws = view(p, workspace);
    WsView gws = ws;                 // redo of failed tensors: own records, gated by the main ones
    gws.sel = reinterpret_cast<TensorSel*>(wb + p->off_gsel);
    gws.gate = ws.sel;
    MultiArgs ma;
    ma.desc = p->d_desc; ma.T = p->T; ma.ntiles = p->ntiles; ma.nstiles = p->nstiles;
    ma.per = mg.per; ma.full_ctas = mg.full;
    ma.pool_cap = std::min<uint32_t>(mg.pool, p->cand_cap / mg.G);     // each CTA's share
    ma.pool_smem_words = (mg.pool + 31) / 32; ma.ntab = mg.ntab;
    ma.small_ids = p->d_small; ma.n_small = (uint32_t)p->small_ids.size(); ma.n_tiny = p->n_tiny;
    ma.reg_ids = p->d_small + p->T; ma.n_reg = (uint32_t)p->reg_ids.size();
    ma.brk = reinterpret_cast<TensorSel*>(wb + p->off_ssel);
    ma.g = grad; ma.r = residual; ma.out_idx = out_idx; ma.out_val = out_val; ma.out_count = out_count;
    ma.cand = reinterpret_cast<uint2*>(wb + p->off_cidx);
    ma.mid = reinterpret_cast<uint2*>(wb + p->off_mmid);
    ma.mid_n = reinterpret_cast<uint32_t*>(wb + p->off_midn);
    ma.shist = reinterpret_cast<uint32_t*>(wb + p->off_shist);
    ma.bhist = reinterpret_cast<uint32_t*>(wb + p->off_bhist);
    ma.tile_cnt = reinterpret_cast<uint32_t*>(wb + p->off_tinfo);
    ma.skeys = reinterpret_cast<uint4*>(wb + p->off_skeys);
    ma.ws = ws; ma.gws = gws;
    ma.cl = clean_args(p, workspace, GC_ROUTE_TOPK_MANY, expect_clean);
    return ma;
}

// Argument block of the many-tensor threshold kernel for one worker's buffers and a given geometry.
static ThrMultiArgs thr_multi_args(const gc_plan_s* p, const MultiGeom& mg, const float* grad, float* residual,
                                   uint32_t* out_idx, float* out_val, uint32_t* out_count, void* workspace) {
    char* wb = static_cast<char*>(workspace);
    ThrMultiArgs ta;
    ta.desc = p->d_desc; ta.T = p->T; ta.ntiles = p->ntiles; ta.nstiles = p->nstiles;
    ta.per = mg.per; ta.pool_cap = mg.pool; ta.ntab = mg.ntab;
    ta.small_ids = p->d_small; ta.n_small = (uint32_t)p->small_ids.size();
    ta.reg_ids = p->d_small + p->T; ta.n_reg = (uint32_t)p->reg_ids.size();
    ta.g = grad; ta.r = residual; ta.out_idx = out_idx; ta.out_val = out_val; ta.out_count = out_count;
    ta.cand = reinterpret_cast<uint2*>(wb + p->off_cidx);
    ta.shist = reinterpret_cast<uint32_t*>(wb + p->off_shist);
    ta.skeys = reinterpret_cast<uint4*>(wb + p->off_skeys);
    ta.tile_cnt = reinterpret_cast<uint32_t*>(wb + p->off_tinfo);
    ta.tsel = reinterpret_cast<TensorSel*>(wb + p->off_ssel);
    ta.ws = view(p, workspace);
    return ta;
}

static int compress_impl(gc_plan_t* p, const void* grad_any, bool bf16, float* residual, uint32_t* out_idx,
                         float* out_val, uint32_t* out_count, void* workspace, void* stream) {
    const float* grad = static_cast<const float*>(grad_any);       // only dereferenced as such when !bf16
    if (p == nullptr) return GC_E_INVALID;
    if (p->device < 0) return GC_E_UNSUPPORTED;
    if (!on_plan_device(p)) return GC_E_INVALID;
    // a bf16 gradient is read by the two fused top-k kernels only
    if (bf16 && !(p->mode == GC_TOPK && p->path == GC_PATH_AUTO && (p->single_grid > 0 || p->multi_grid > 0)))
        return GC_E_UNSUPPORTED;
    if (p->total_n == 0) return GC_OK;
    if (grad == nullptr || residual == nullptr || out_idx == nullptr || out_val == nullptr ||
        workspace == nullptr)
        return GC_E_INVALID;
    if ((reinterpret_cast<uintptr_t>(grad) & 15u) || (reinterpret_cast<uintptr_t>(residual) & 15u) ||
        (reinterpret_cast<uintptr_t>(workspace) & 255u) || (reinterpret_cast<uintptr_t>(out_idx) & 3u) ||
        (reinterpret_cast<uintptr_t>(out_val) & 3u))
        return GC_E_INVALID;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    WsView ws = view(p, workspace);
    const int route = compress_route(p);
    // The one-tensor top-k kernel leaves the control block as the next launch needs it; when the
    // caller has promised that nobody else touches the workspace, the clearing launch is skipped
    // for a workspace that kernel ran on last (the kernel checks a mark in the header and leaves
    // with GC_E_INVALID if the promise was broken).
    const bool self_cleaning = route == GC_ROUTE_TOPK_ONE || route == GC_ROUTE_TOPK_MANY;
    const bool kept_clean = take_clean(p, workspace) && p->ws_private && self_cleaning;
    if (!kept_clean) {
        Timed tm(p, s, GC_K_CLEAR_CTRL);
        const size_t n16 = p->control_bytes / 16;             // control_bytes is a multiple of 256
        const int gc = (int)std::min<size_t>((n16 + kBlock - 1) / kBlock, (size_t)p->sm_count * 8);
        k_clear<<<gc, kBlock, 0, s>>>(reinterpret_cast<uint4*>(workspace), n16);
    }
    if (out_count != nullptr && p->n_empty > 0) {       // every tensor with elements gets its counts written
        Timed tm(p, s, GC_K_CLEAR_CTRL);
        GC_CUDA(p, cudaMemsetAsync(out_count, 0, sizeof(uint32_t) * 2 * (size_t)p->T, s));
    }
    const uint32_t nt = p->ntiles;
    const int gh = (int)std::min<uint32_t>(nt, (uint32_t)p->grid_hist);
    const int gcp = (int)std::min<uint32_t>(nt, (uint32_t)p->grid_compact);
    char* wb = static_cast<char*>(workspace);
    if (route == GC_ROUTE_THRESHOLD_ONE) {
        // one large tensor: sample, exact threshold, fold + hits and emission in one cooperative launch
        ThrSingleArgs ta;
        ta.d = p->desc[0]; ta.desc = p->d_desc; ta.ntiles = nt; ta.maxt = p->thr_maxt; ta.pool_cap = p->thr_pool;
        ta.sample_rounds = p->thr_rounds;
        ta.g = grad; ta.r = residual; ta.out_idx = out_idx; ta.out_val = out_val; ta.out_count = out_count;
        ta.cand = reinterpret_cast<uint2*>(wb + p->off_cidx);
        ta.skeys = reinterpret_cast<uint4*>(wb + p->off_skeys);
        ta.hist5 = reinterpret_cast<uint32_t*>(wb + p->off_hist5);
        ta.hist13 = ta.hist5 + 2 * kHistBins;          // slots 2..5 of the six
        ta.mid = reinterpret_cast<uint2*>(wb + p->off_mid); ta.mid_cap = (uint32_t)kSingleMidCap;
        ta.fine = reinterpret_cast<uint32_t*>(wb + p->off_fine);
        ta.tile_cnt = reinterpret_cast<uint32_t*>(wb + p->off_tinfo);
        ta.seg_tot = reinterpret_cast<uint32_t*>(wb + p->off_rowseg);
        ta.ws = ws;
        void* args[] = {&ta};
        Timed tm(p, s, GC_K_FUSED);
        GC_CUDA(p, cudaLaunchCooperativeKernel((const void*)k_threshold_single, dim3(p->thr_grid), dim3(kBlock),
                                               args, p->thr_smem, s));
        return GC_OK;
    }
    if (route == GC_ROUTE_THRESHOLD_MANY) {
        // several tensors: sample, exact thresholds, fold + hits and emission in one cooperative launch
        MultiGeom mg;
        mg.G = p->thrm_grid; mg.per = p->thrm_per; mg.pool = p->thrm_pool; mg.ntab = p->thrm_ntab; mg.smem = p->thrm_smem;
        ThrMultiArgs ta = thr_multi_args(p, mg, grad, residual, out_idx, out_val, out_count, workspace);
        void* args[] = {&ta};
        Timed tm(p, s, GC_K_FUSED);
        GC_CUDA(p, cudaLaunchCooperativeKernel((const void*)k_threshold_multi, dim3(p->thrm_grid), dim3(kBlock),
                                               args, p->thrm_smem, s));
        return GC_OK;
    }
    if (route == GC_ROUTE_THRESHOLD_STAGED) {
        // exact order statistic of the sample (three radix levels), then one fused pass
        WsView sws = ws;
        sws.sel = reinterpret_cast<TensorSel*>(wb + p->off_ssel);
        const int gs = (int)std::min<uint32_t>(p->nstiles, (uint32_t)p->grid_sample);
        { Timed tm(p, s, GC_K_SAMPLE);
          k_hist<0, SRC_SAMPLE><<<gs, kBlock, 0, s>>>(p->d_desc, p->T, p->nstiles, grad, residual, sws); }
        { Timed tm(p, s, GC_K_SAMPLE);
          k_hist<1, SRC_SAMPLE><<<gs, kBlock, 0, s>>>(p->d_desc, p->T, p->nstiles, grad, residual, sws); }
        { Timed tm(p, s, GC_K_SAMPLE);
          k_hist<2, SRC_SAMPLE><<<gs, kBlock, 0, s>>>(p->d_desc, p->T, p->nstiles, grad, residual, sws); }
        { Timed tm(p, s, GC_K_THRESHOLD_EMIT);
          const int gt = (int)std::min<uint32_t>(nt, (uint32_t)p->grid_thr);
          k_threshold_emit<<<gt, kBlock, 0, s>>>(p->d_desc, p->T, nt, grad, residual, out_idx, out_val,
                                                 out_count, ws, sws.sel, 0); }
        GC_CUDA(p, cudaGetLastError());
        return GC_OK;
    }
    if (route == GC_ROUTE_EXACT) {
        // exact multi-pass path on its own: fold + three histogram levels + ordered compaction
        { Timed tm(p, s, GC_K_FOLD_HIST);
          k_hist<0, SRC_FOLD><<<gh, kBlock, 0, s>>>(p->d_desc, p->T, nt, grad, residual, ws); }
        { Timed tm(p, s, GC_K_HIST_REFINE);
          k_hist<1, SRC_RESID><<<gh, kBlock, 0, s>>>(p->d_desc, p->T, nt, nullptr, residual, ws); }
        { Timed tm(p, s, GC_K_HIST_REFINE);
          k_hist<2, SRC_RESID><<<gh, kBlock, 0, s>>>(p->d_desc, p->T, nt, nullptr, residual, ws); }
        { Timed tm(p, s, GC_K_COMPACT);
          k_compact<<<gcp, kBlock, 0, s>>>(p->d_desc, p->T, nt, residual, out_idx, out_val, out_count, ws, 0); }
        GC_CUDA(p, cudaGetLastError());
        return GC_OK;
    }
    // candidate path: sample -> fold + candidates -> refine on candidates -> compaction from
    // candidates; then the exact kernels, gated to the tensors (normally none) it gave up on
    WsView sws = ws;                 // sample select works on its own records
    sws.sel = reinterpret_cast<TensorSel*>(wb + p->off_ssel);
    WsView gws = ws;                 // redo of failed tensors: own records, gated by the main ones
    gws.sel = reinterpret_cast<TensorSel*>(wb + p->off_gsel);
    gws.gate = ws.sel;
    CandView cv;
    cv.pair = reinterpret_cast<uint2*>(wb + p->off_cidx);
    cv.chunk_info = reinterpret_cast<uint2*>(wb + p->off_tinfo);
    cv.group_cnt = reinterpret_cast<unsigned long long*>(wb + p->off_gstate);
    cv.cap = p->cand_cap;
    cv.ssel = sws.sel;
    if (route == GC_ROUTE_TOPK_ONE) {
        // one large tensor: candidates stay in shared memory
        SingleArgs sa;
        sa.d = p->desc[0]; sa.desc = p->d_desc; sa.ntiles = nt; sa.maxt = p->single_maxt; sa.rows = p->single_rows;
        sa.pool_cap = std::min<uint32_t>(p->single_pool, p->cand_cap);
        sa.cand = reinterpret_cast<uint2*>(wb + p->off_cidx);
        sa.g = grad_any; sa.r = residual; sa.out_idx = out_idx; sa.out_val = out_val; sa.out_count = out_count;
        sa.hist5 = reinterpret_cast<uint32_t*>(wb + p->off_hist5);
        sa.srank_hi = p->single_srank_hi; sa.srank_mid = p->single_srank_mid; sa.mid_cap = (uint32_t)kSingleMidCap;
        sa.mid = reinterpret_cast<uint2*>(wb + p->off_mid);
        sa.fine = reinterpret_cast<uint32_t*>(wb + p->off_fine);
        sa.age = reinterpret_cast<uint32_t*>(wb + p->off_age);
        sa.tile_cnt = reinterpret_cast<uint32_t*>(wb + p->off_tinfo);
        sa.seg_tot = reinterpret_cast<uint32_t*>(wb + p->off_rowseg);
        sa.ws = ws; sa.gws = gws;
        sa.cl = clean_args(p, workspace, GC_ROUTE_TOPK_ONE, kept_clean);
        note_clean(p, workspace);
        void* args[] = {&sa};
        Timed tm(p, s, GC_K_FUSED);
        const void* kfn = bf16 ? (const void*)k_topk_single<GradBF16> : (const void*)k_topk_single<GradF32>;
        GC_CUDA(p, cudaLaunchCooperativeKernel(kfn, dim3(p->single_grid), dim3(kBlock), args, p->single_smem, s));
        return GC_OK;
    }
    if (route == GC_ROUTE_TOPK_MANY) {
        // many tensors: one cooperative launch, four grid barriers
        MultiGeom mg;
        mg.G = p->multi_grid; mg.per = p->multi_per; mg.pool = p->multi_pool; mg.full = p->multi_full;
        mg.ntab = p->multi_ntab; mg.smem = p->multi_smem;
        MultiArgs ma = multi_args(p, mg, grad_any, residual, out_idx, out_val, out_count, workspace, kept_clean);
        note_clean(p, workspace);
        void* args[] = {&ma};
        Timed tm(p, s, GC_K_FUSED);
        const void* kfn = bf16 ? (const void*)k_topk_multi<GradBF16> : (const void*)k_topk_multi<GradF32>;
        GC_CUDA(p, cudaLaunchCooperativeKernel(kfn, dim3(p->multi_grid), dim3(kBlock), args, p->multi_smem, s));
        return GC_OK;
    }
    if (route == GC_ROUTE_TOPK_GENERAL) {
        // everything in one cooperative launch
        FusedArgs fa;
        fa.desc = p->d_desc; fa.T = p->T; fa.ntiles = nt; fa.nstiles = p->nstiles; fa.ngroups = p->ngroups;
        fa.small_ids = p->d_small; fa.n_small = (uint32_t)p->small_ids.size();
        fa.g = grad; fa.r = residual; fa.out_idx = out_idx; fa.out_val = out_val; fa.out_count = out_count;
        fa.ws = ws; fa.sws = sws; fa.gws = gws; fa.cv = cv;
        void* args[] = {&fa};
        const uint32_t want = std::max<uint32_t>(std::max<uint32_t>(nt, p->nstiles), 1u);   // nt >= #small tensors
        const int gf = (int)std::min<uint32_t>(want, (uint32_t)p->grid_fused);
        Timed tm(p, s, GC_K_FUSED);
        GC_CUDA(p, cudaLaunchCooperativeKernel((const void*)k_compress_fused, dim3(gf), dim3(kBlock), args, 0, s));
        return GC_OK;
    }
    if (!p->small_ids.empty()) {
        Timed tm(p, s, GC_K_SMALL);
        const int gsm = (int)std::min<uint32_t>((uint32_t)p->small_ids.size(), (uint32_t)p->grid_hist);
        k_small_tensors<<<gsm, kBlock, 0, s>>>(p->d_desc, p->T, p->d_small, (uint32_t)p->small_ids.size(), grad,
                                               residual, out_idx, out_val, out_count);
    }
    if (p->nstiles > 0) {
        const int gs = (int)std::min<uint32_t>(p->nstiles, (uint32_t)p->grid_sample);
        // two radix levels on the sample: tau_lo is the exact srank-th sampled key cut to 21 bits,
        // so the size of the candidate set is binomial whatever the shape of the distribution
        { Timed tm(p, s, GC_K_SAMPLE);
          k_hist<0, SRC_SAMPLE><<<gs, kBlock, 0, s>>>(p->d_desc, p->T, p->nstiles, grad, residual, sws); }
        { Timed tm(p, s, GC_K_SAMPLE);
          k_hist<1, SRC_SAMPLE><<<gs, kBlock, 0, s>>>(p->d_desc, p->T, p->nstiles, grad, residual, sws); }
    }
    { Timed tm(p, s, GC_K_FOLD_CAND);
      const int gf = (int)std::min<uint32_t>(nt, (uint32_t)p->grid_fold);
      k_fold_cand<<<gf, kBlock, 0, s>>>(p->d_desc, p->T, nt, grad, residual, ws, cv); }
    {
        const int gch = (int)std::min<uint32_t>((nt + 2 * kWarps - 1) / (2 * kWarps), (uint32_t)p->grid_chist);
        { Timed tm(p, s, GC_K_CAND_REFINE);
          k_cand_hist<1><<<gch, kBlock, 0, s>>>(p->d_desc, p->T, nt, ws, cv); }
        { Timed tm(p, s, GC_K_CAND_REFINE);
          k_cand_hist<2><<<gch, kBlock, 0, s>>>(p->d_desc, p->T, nt, ws, cv); }
    }
    {
        const int gcc = (int)std::min<uint32_t>(p->ngroups, (uint32_t)p->grid_ccompact);
        { Timed tm(p, s, GC_K_CAND_COMPACT);
          k_cand_compact<false><<<gcc, kBlock, 0, s>>>(p->d_desc, p->T, p->ngroups, residual, out_idx, out_val,
                                                       out_count, ws, cv); }
        { Timed tm(p, s, GC_K_CAND_COMPACT);
          k_cand_compact<true><<<gcc, kBlock, 0, s>>>(p->d_desc, p->T, p->ngroups, residual, out_idx, out_val,
                                                      out_count, ws, cv); }
    }
    {
        { Timed tm(p, s, GC_K_HIST_REFINE);
          const int gr = (int)std::min<uint32_t>((nt + kWarps - 1) / kWarps, (uint32_t)p->grid_chist);
          k_cand_restore<<<gr, kBlock, 0, s>>>(p->d_desc, p->T, nt, residual, ws, cv); }
        { Timed tm(p, s, GC_K_HIST_REFINE);
          k_hist<0, SRC_RESID><<<gh, kBlock, 0, s>>>(p->d_desc, p->T, nt, nullptr, residual, gws); }
        { Timed tm(p, s, GC_K_HIST_REFINE);
          k_hist<1, SRC_RESID><<<gh, kBlock, 0, s>>>(p->d_desc, p->T, nt, nullptr, residual, gws); }
        { Timed tm(p, s, GC_K_HIST_REFINE);
          k_hist<2, SRC_RESID><<<gh, kBlock, 0, s>>>(p->d_desc, p->T, nt, nullptr, residual, gws); }
        { Timed tm(p, s, GC_K_COMPACT);
          k_compact<<<gcp, kBlock, 0, s>>>(p->d_desc, p->T, nt, residual, out_idx, out_val, out_count, gws, 0); }
    }
    GC_CUDA(p, cudaGetLastError());
    return GC_OK;
}

int gc_compress(gc_plan_t* p, const float* grad, float* residual, uint32_t* out_idx, float* out_val,
                uint32_t* out_count, void* workspace, void* stream) {
    return compress_impl(p, grad, false, residual, out_idx, out_val, out_count, workspace, stream);
}

int gc_compress_bf16(gc_plan_t* p, const void* grad_bf16, float* residual, uint32_t* out_idx, float* out_val,
                     uint32_t* out_count, void* workspace, void* stream) {
    return compress_impl(p, grad_bf16, true, residual, out_idx, out_val, out_count, workspace, stream);
}

int gc_compress_workers(gc_plan_t* p, uint32_t W, const float* const* grads, float* const* residuals,
                        uint32_t* const* out_idx, float* const* out_val, uint32_t* const* out_count,
                        void* const* workspaces, void* stream) {
    if (p == nullptr) return GC_E_INVALID;
    if (W > GC_MAX_WORKERS) return GC_E_TOO_LARGE;
    if (p->device < 0) return GC_E_UNSUPPORTED;
    if (!on_plan_device(p)) return GC_E_INVALID;
    if (W == 0 || p->total_n == 0) return GC_OK;
    if (grads == nullptr || residuals == nullptr || out_idx == nullptr || out_val == nullptr || workspaces == nullptr)
        return GC_E_INVALID;
    for (uint32_t w = 0; w < W; ++w) {
        if (grads[w] == nullptr || residuals[w] == nullptr || out_idx[w] == nullptr || out_val[w] == nullptr ||
            workspaces[w] == nullptr || (out_count != nullptr && out_count[w] == nullptr))
            return GC_E_INVALID;
        if ((reinterpret_cast<uintptr_t>(grads[w]) & 15u) || (reinterpret_cast<uintptr_t>(residuals[w]) & 15u) ||
            (reinterpret_cast<uintptr_t>(workspaces[w]) & 255u) || (reinterpret_cast<uintptr_t>(out_idx[w]) & 3u) ||
            (reinterpret_cast<uintptr_t>(out_val[w]) & 3u))
            return GC_E_INVALID;
        for (uint32_t v = 0; v < w; ++v)         // the calls run at the same time: nothing may be shared
            if (workspaces[v] == workspaces[w] || residuals[v] == residuals[w] || out_idx[v] == out_idx[w] ||
                out_val[v] == out_val[w])
                return GC_E_INVALID;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // how many workers one launch takes: the resident CTAs are dealt out evenly, and a worker's
    // share must still satisfy the kernel's limits (tiles and candidates per CTA)
    uint32_t batch = 0;
    MultiGeom mg;
    const bool topk_multi = p->mode == GC_TOPK && p->path == GC_PATH_AUTO && p->multi_grid > 0;
    const bool thr_multi = p->mode == GC_THRESHOLD && p->path == GC_PATH_AUTO && p->thrm_grid > 0;
    if ((topk_multi || thr_multi) && W >= 2) {
        if (p->wk_W != W) {                      // (kept for the next call; options that change the layout reset it)
            p->wk_W = W; p->wk_batch = 0;
            for (uint32_t wb = std::min<uint32_t>(W, kWorkersPerLaunch); wb >= 2 && p->wk_batch == 0; --wb) {
                const MultiGeom g2 = topk_multi ? multi_geometry(p, (uint32_t)p->grid_multi_max / wb, false)
                                                : thr_multi_geometry(p, (uint32_t)p->grid_thr_multi_max / wb);
                if (g2.G > 0 && g2.smem <= (topk_multi ? p->multi_smem_max : p->thrm_smem_max)) {
                    p->wk_batch = wb; p->wk_geom = g2;
                }
            }
        }
        batch = p->wk_batch; mg = p->wk_geom;
    }
    if (batch == 0) {                            // no shared launch for this plan: one call per worker
        for (uint32_t w = 0; w < W; ++w) {
            const int rc = compress_impl(p, grads[w], false, residuals[w], out_idx[w], out_val[w],
                                         out_count ? out_count[w] : nullptr, workspaces[w], stream);
            if (rc < 0) return rc;
        }
        return GC_OK;
    }
    for (uint32_t w0 = 0; w0 < W; w0 += batch) {
        const uint32_t wn = std::min<uint32_t>(batch, W - w0);
        if (wn == 1) {                           // a lone leftover worker takes the whole device
            const int rc = compress_impl(p, grads[w0], false, residuals[w0], out_idx[w0], out_val[w0],
                                         out_count ? out_count[w0] : nullptr, workspaces[w0], stream);
            if (rc < 0) return rc;
            continue;
        }
        ClearMany cm;
        WorkersArgs wa;
        ThrWorkersArgs ta;
        wa.W = ta.W = wn; wa.G = ta.G = mg.G;
        // the clearing launch is skipped only if every workspace of this launch was left clean
        bool kept_clean = p->ws_private && topk_multi;
        for (uint32_t i = 0; i < wn; ++i) kept_clean = take_clean(p, workspaces[w0 + i]) && kept_clean;
        for (uint32_t i = 0; i < wn; ++i) {
            const uint32_t w = w0 + i;
            cm.p[i] = reinterpret_cast<uint4*>(workspaces[w]);
            uint32_t* const oc = out_count ? out_count[w] : nullptr;
            if (topk_multi) {
                wa.per[i] = multi_args(p, mg, grads[w], residuals[w], out_idx[w], out_val[w], oc, workspaces[w], kept_clean);
                note_clean(p, workspaces[w]);
            }
            if (!topk_multi) ta.per[i] = thr_multi_args(p, mg, grads[w], residuals[w], out_idx[w], out_val[w], oc, workspaces[w]);
            if (oc != nullptr && p->n_empty > 0) {
                Timed tm(p, s, GC_K_CLEAR_CTRL);
                GC_CUDA(p, cudaMemsetAsync(oc, 0, sizeof(uint32_t) * 2 * (size_t)p->T, s));
            }
        }
        for (uint32_t i = wn; i < kWorkersPerLaunch; ++i) {
            cm.p[i] = nullptr;
            if (topk_multi) wa.per[i] = wa.per[0]; else ta.per[i] = ta.per[0];
        }
        if (!kept_clean) {
            Timed tm(p, s, GC_K_CLEAR_CTRL);
            const size_t n16 = p->control_bytes / 16;
            const unsigned gx = (unsigned)std::min<size_t>((n16 + kBlock - 1) / kBlock, (size_t)p->sm_count * 8 / wn + 1);
            k_clear_many<<<dim3(gx, wn), kBlock, 0, s>>>(cm, n16);
        }
        void* args[] = {topk_multi ? (void*)&wa : (void*)&ta};
        Timed tm(p, s, GC_K_FUSED);
        GC_CUDA(p, cudaLaunchCooperativeKernel(topk_multi ? (const void*)k_topk_workers<GradF32> : (const void*)k_threshold_workers,
                                               dim3(mg.G * wn), dim3(kBlock), args, mg.smem, s));
    }
    return GC_OK;
}

int gc_decompress_accumulate(gc_plan_t* p, uint32_t W, const uint32_t* const* idx,
                             const float* const* val, const uint32_t* const* count,
                             float* dense_out, int zero_first, void* workspace, void* stream) {
    if (p == nullptr) return GC_E_INVALID;
    if (W > GC_MAX_WORKERS) return GC_E_TOO_LARGE;
    if (p->device < 0) return GC_E_UNSUPPORTED;
    if (!on_plan_device(p)) return GC_E_INVALID;
    if (p->total_n == 0) return GC_OK;
    if (dense_out == nullptr || workspace == nullptr) return GC_E_INVALID;
    if (W > 0 && (idx == nullptr || val == nullptr)) return GC_E_INVALID;
    for (uint32_t w = 0; w < W; ++w) {
        if (idx[w] == nullptr || val[w] == nullptr) return GC_E_INVALID;
        if (count != nullptr && count[w] == nullptr) return GC_E_INVALID;
    }
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return GC_E_INVALID;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    WsView ws = view(p, workspace);
    // few workers per tile: overlap the tile's way out with the next tile -- unless a CTA has so few
    // tiles that twice the CTAs with one buffer each are through sooner (25.6M elements: 21.0 against
    // 22.6 us; 50M: 39.3 against 37.4 us)
    const uint32_t ntl_all = (uint32_t)((p->total_n + kDecTile - 1) / kDecTile);
    const int nbuf = (W <= 2 && p->grid_decode[1] > 0 && ntl_all >= 10u * (uint32_t)p->grid_decode[1]) ? 2 : 1;
    if ((count == nullptr || p->T == 1) && W > 0 && p->total_cap > 0 && p->path != GC_PATH_EXACT &&
        p->grid_decode[nbuf - 1] > 0) {
        // every list is one run of pairs in ascending index (total_cap of them, or - one-tensor plans
        // with count arrays - as many as the list's first count says): tiled decode, dense buffer
        // written once (and not read at all when it is cleared first)
        DecodeLists ls;
        for (uint32_t w = 0; w < 64; ++w) {
            ls.idx[w] = idx[w < W ? w : 0]; ls.val[w] = val[w < W ? w : 0];
            ls.len[w] = count != nullptr ? count[w < W ? w : 0] : nullptr;
        }
        const uint32_t ntl = (uint32_t)((p->total_n + kDecTile - 1) / kDecTile);
        const int grid = (int)std::min<uint32_t>(ntl, (uint32_t)p->grid_decode[nbuf - 1]);
        const int use_bulk = (reinterpret_cast<uintptr_t>(dense_out) & 15u) == 0 ? 1 : 0;
        Timed tm(p, s, GC_K_DECODE_TILES);
        const DecodeRoute rt = decode_route<false>(p, W, zero_first != 0);
        if (rt.wide) {
            auto kw = rt.any ? k_decode_any<false> : k_decode_wide<false>;
            kw<<<(int)std::min<uint32_t>(ntl, (uint32_t)rt.grid), kDecBlock, rt.smem, s>>>(
                ls, W, (uint32_t)p->total_cap, (uint32_t)p->total_n, dense_out, zero_first ? 1 : 0, use_bulk, rt.win,
                ws.hdr, ApplyArgs{});
            GC_CUDA(p, cudaGetLastError());
            return GC_OK;
        }
        if (rt.rounds != kDecRounds)
            k_decode_tiles<false, 2 * kDecRounds><<<(int)std::min<uint32_t>(ntl, (uint32_t)p->grid_decode8), kDecBlock,
                                                    kDecTileBytes, s>>>(ls, W, (uint32_t)p->total_cap, (uint32_t)p->total_n,
                                                                        dense_out, zero_first ? 1 : 0, use_bulk, 1, ws.hdr,
                                                                        ApplyArgs{});
        else
            k_decode_tiles<false, kDecRounds><<<grid, kDecBlock, nbuf * kDecTileBytes, s>>>(
                ls, W, (uint32_t)p->total_cap, (uint32_t)p->total_n, dense_out, zero_first ? 1 : 0, use_bulk, nbuf, ws.hdr,
                ApplyArgs{});
        GC_CUDA(p, cudaGetLastError());
        return GC_OK;
    }
    if (count != nullptr && p->T > 1 && W > 0 && p->total_cap > 0 && p->path != GC_PATH_EXACT &&
        p->grid_decode_seg[nbuf - 1] > 0 && p->d_dectile != nullptr) {
        // lists with per-tensor counts: ascending inside a tensor, unused slots between tensors --
        // the same tile loop, cut at the tensor boundaries
        DecodeLists ls;
        for (uint32_t w = 0; w < 64; ++w) {
            ls.idx[w] = idx[w < W ? w : 0]; ls.val[w] = val[w < W ? w : 0]; ls.len[w] = count[w < W ? w : 0];
        }
        const uint32_t ntl = (uint32_t)((p->total_n + kDecTile - 1) / kDecTile);
        const int grid = (int)std::min<uint32_t>(ntl, (uint32_t)p->grid_decode_seg[nbuf - 1]);
        const int use_bulk = (reinterpret_cast<uintptr_t>(dense_out) & 15u) == 0 ? 1 : 0;
        Timed tm(p, s, GC_K_DECODE_TILES);
        k_decode_segments<false><<<grid, kDecBlock, nbuf * kDecTileBytes, s>>>(
            ls, W, p->d_desc, p->T, p->d_dectile, (uint32_t)p->total_n, dense_out, zero_first ? 1 : 0, use_bulk, nbuf,
            ws.hdr, ApplyArgs{});
        GC_CUDA(p, cudaGetLastError());
        return GC_OK;
    }
    if (zero_first) {
        Timed tm(p, s, GC_K_DECODE_CLEAR);
        GC_CUDA(p, cudaMemsetAsync(dense_out, 0, sizeof(float) * (size_t)p->total_n, s));
    }
    if (p->total_cap == 0) return GC_OK;
    const uint32_t cap = (uint32_t)p->total_cap;
    const int grid = (int)((cap + 255u) / 256u);
    for (uint32_t w = 0; w < W; ++w) {
        Timed tm(p, s, GC_K_DECODE_ADD);
        k_scatter_add<<<grid, 256, 0, s>>>(p->d_desc, p->T, cap, (uint32_t)p->total_n, idx[w], val[w],
                                           count ? count[w] : nullptr, dense_out, ws.hdr);
    }
    GC_CUDA(p, cudaGetLastError());
    return GC_OK;
}

int gc_decompress_apply_momentum(gc_plan_t* p, uint32_t W, const uint32_t* const* idx, const float* const* val,
                                 const uint32_t* const* count, float* param, float* velocity, float lr,
                                 float momentum, float scale, void* workspace, void* stream) {
    if (p == nullptr) return GC_E_INVALID;
    if (W > GC_MAX_WORKERS) return GC_E_TOO_LARGE;
    if (p->device < 0) return GC_E_UNSUPPORTED;
    if (!on_plan_device(p)) return GC_E_INVALID;
    if (p->total_n == 0) return GC_OK;
    if (param == nullptr || velocity == nullptr || workspace == nullptr) return GC_E_INVALID;
    if (W > 0 && (idx == nullptr || val == nullptr)) return GC_E_INVALID;
    for (uint32_t w = 0; w < W; ++w) {
        if (idx[w] == nullptr || val[w] == nullptr) return GC_E_INVALID;
        if (count != nullptr && count[w] == nullptr) return GC_E_INVALID;
    }
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) || (reinterpret_cast<uintptr_t>(param) & 15u) ||
        (reinterpret_cast<uintptr_t>(velocity) & 15u))
        return GC_E_INVALID;
    const bool segmented = count != nullptr && p->T != 1;              // lists with unused slots between tensors
    if ((segmented ? p->grid_decode_seg_apply : p->grid_decode[0]) <= 0) return GC_E_UNSUPPORTED;
    if (segmented && p->d_dectile == nullptr) return GC_E_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    WsView ws = view(p, workspace);
    DecodeLists ls;
    for (uint32_t w = 0; w < 64; ++w) {
        const uint32_t q = w < W ? w : 0;
        ls.idx[w] = W ? idx[q] : nullptr; ls.val[w] = W ? val[q] : nullptr;
        ls.len[w] = (W && count != nullptr) ? count[q] : nullptr;
    }
    const uint32_t ntl = (uint32_t)((p->total_n + kDecTile - 1) / kDecTile);
    const int grid = (int)std::min<uint32_t>(ntl, (uint32_t)p->grid_decode[0]);
    ApplyArgs ap{param, velocity, lr, momentum, scale};
    Timed tm(p, s, GC_K_DECODE_TILES);
    if (segmented && W > 0) {
        k_decode_segments<true><<<(int)std::min<uint32_t>(ntl, (uint32_t)p->grid_decode_seg_apply), kDecBlock,
                                  kDecTileBytes, s>>>(ls, W, p->d_desc, p->T, p->d_dectile, (uint32_t)p->total_n,
                                                      nullptr, 1, 0, 1, ws.hdr, ap);
        GC_CUDA(p, cudaGetLastError());
        return GC_OK;
    }
    const DecodeRoute rt = decode_route<true>(p, W, true);
    if (rt.wide) {
        auto kw = rt.any ? k_decode_any<true> : k_decode_wide<true>;
        kw<<<(int)std::min<uint32_t>(ntl, (uint32_t)rt.grid), kDecBlock, rt.smem, s>>>(
            ls, W, (uint32_t)p->total_cap, (uint32_t)p->total_n, nullptr, 1, 0, rt.win, ws.hdr, ap);
        GC_CUDA(p, cudaGetLastError());
        return GC_OK;
    }
    if (rt.rounds != kDecRounds && p->grid_decode8_apply > 0)
        k_decode_tiles<true, 2 * kDecRounds><<<(int)std::min<uint32_t>(ntl, (uint32_t)p->grid_decode8_apply), kDecBlock,
                                               kDecTileBytes, s>>>(ls, W, (uint32_t)p->total_cap, (uint32_t)p->total_n,
                                                                   nullptr, 1, 0, 1, ws.hdr, ap);
    else
        k_decode_tiles<true, kDecRounds><<<grid, kDecBlock, kDecTileBytes, s>>>(
            ls, W, (uint32_t)p->total_cap, (uint32_t)p->total_n, nullptr, 1, 0, 1, ws.hdr, ap);
    GC_CUDA(p, cudaGetLastError());
    return GC_OK;
}

int gc_last_status(gc_plan_t* p, const void* workspace, void* stream, int32_t* status, uint64_t* detail) {
    if (p == nullptr || workspace == nullptr || status == nullptr) return GC_E_INVALID;
    if (p->device < 0) return GC_E_UNSUPPORTED;
    if (!on_plan_device(p)) return GC_E_INVALID;
    WsHeader h;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    GC_CUDA(p, cudaMemcpyAsync(&h, workspace, sizeof(WsHeader), cudaMemcpyDeviceToHost, s));
    GC_CUDA(p, cudaStreamSynchronize(s));
    *status = h.status;
    if (detail) *detail = h.detail;
    if (h.status < 0) (void)take_clean(p, workspace);    // a failed launch leaves no clean block behind
    return GC_OK;
}

int gc_compress_host(gc_plan_t* p, const float* host_grad, float* grad_staging, float* residual,
                     uint32_t* out_idx, float* out_val, uint32_t* out_count, uint32_t* host_idx,
                     float* host_val, void* workspace, void* stream) {
    if (p == nullptr) return GC_E_INVALID;
    if (p->device < 0) return GC_E_UNSUPPORTED;
    if (!on_plan_device(p)) return GC_E_INVALID;
    if (p->total_n == 0) return GC_OK;
    if (host_grad == nullptr || grad_staging == nullptr || host_idx == nullptr || host_val == nullptr)
        return GC_E_INVALID;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    gc_plan_s::StagingUse* use = nullptr;
    if (!p->recs.empty()) {
        // per-kernel timing is on: everything on the caller's stream, bracketed by its events
        Timed tm(p, s, GC_K_COPY);
        GC_CUDA(p, cudaMemcpyAsync(grad_staging, host_grad, sizeof(float) * (size_t)p->total_n,
                                   cudaMemcpyHostToDevice, s));
    } else {
        if (p->copy_stream == nullptr) {
            GC_CUDA(p, cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking));
            GC_CUDA(p, cudaEventCreateWithFlags(&p->ev_copied, cudaEventDisableTiming));
        }
        for (auto& u : p->staging) if (u.ptr == grad_staging) use = &u;
        if (use == nullptr) {
            // first call with this staging buffer: whatever the caller's stream still does with it comes first
            if (p->staging.size() >= 8) {                // (callers rotate two or three buffers)
                for (auto& u : p->staging) cudaEventDestroy(u.done);
                p->staging.clear();
            }
            gc_plan_s::StagingUse u{grad_staging, nullptr};
            GC_CUDA(p, cudaEventCreateWithFlags(&u.done, cudaEventDisableTiming));
            p->staging.push_back(u);
            use = &p->staging.back();
            GC_CUDA(p, cudaEventRecord(use->done, s));
        }
        GC_CUDA(p, cudaStreamWaitEvent(p->copy_stream, use->done, 0));      // the compress that last read the buffer
        GC_CUDA(p, cudaMemcpyAsync(grad_staging, host_grad, sizeof(float) * (size_t)p->total_n,
                                   cudaMemcpyHostToDevice, p->copy_stream));
        GC_CUDA(p, cudaEventRecord(p->ev_copied, p->copy_stream));
        GC_CUDA(p, cudaStreamWaitEvent(s, p->ev_copied, 0));
    }
    int rc = gc_compress(p, grad_staging, residual, out_idx, out_val, out_count, workspace, stream);
    if (rc < 0) return rc;
    if (use != nullptr) GC_CUDA(p, cudaEventRecord(use->done, s));          // the staging buffer may be refilled
    {
        Timed tm(p, s, GC_K_COPY);
        GC_CUDA(p, cudaMemcpyAsync(host_idx, out_idx, sizeof(uint32_t) * (size_t)p->total_cap,
                                   cudaMemcpyDeviceToHost, s));
    }
    {
        Timed tm(p, s, GC_K_COPY);
        GC_CUDA(p, cudaMemcpyAsync(host_val, out_val, sizeof(float) * (size_t)p->total_cap,
                                   cudaMemcpyDeviceToHost, s));
    }
    return rc;
}

int gc_profile_enable(gc_plan_t* p, uint32_t max_records) {
    if (p == nullptr) return GC_E_INVALID;
    if (p->device < 0) return GC_E_UNSUPPORTED;
    for (auto& r : p->recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    p->recs.clear();
    p->recs_used = 0;
    p->recs.reserve(max_records);
    for (uint32_t i = 0; i < max_records; ++i) {
        gc_plan_s::Rec r{};
        cudaError_t e = cudaEventCreate(&r.a);
        if (e == cudaSuccess) e = cudaEventCreate(&r.b);
        if (e != cudaSuccess) { p->last_cuda_error = (int)e; (void)cudaGetLastError(); return GC_E_CUDA; }
        p->recs.push_back(r);
    }
    return GC_OK;
}

int gc_profile_read(gc_plan_t* p, float* total_ms, uint32_t* launches) {
    if (p == nullptr || total_ms == nullptr || launches == nullptr) return GC_E_INVALID;
    if (p->device < 0) return GC_E_UNSUPPORTED;
    for (int i = 0; i < GC_K_COUNT; ++i) { total_ms[i] = 0.f; launches[i] = 0; }
    GC_CUDA(p, cudaDeviceSynchronize());
    for (size_t i = 0; i < p->recs_used; ++i) {
        float ms = 0.f;
        GC_CUDA(p, cudaEventElapsedTime(&ms, p->recs[i].a, p->recs[i].b));
        int id = p->recs[i].id;
        if (id < 0 || id >= GC_K_COUNT) id = GC_K_OTHER;
        total_ms[id] += ms;
        launches[id] += 1;
    }
    p->recs_used = 0;
    return GC_OK;
}

const char* gc_kernel_name(int id) {
    switch (id) {
        case GC_K_CLEAR_CTRL: return "clear_ctrl";
        case GC_K_FOLD_HIST: return "fold_hist";
        case GC_K_HIST_REFINE: return "hist_refine";
        case GC_K_COMPACT: return "compact";
        case GC_K_DECODE_CLEAR: return "decode_clear";
        case GC_K_DECODE_ADD: return "decode_add";
        case GC_K_COPY: return "copy";
        case GC_K_SAMPLE: return "sample";
        case GC_K_THRESHOLD_EMIT: return "threshold_emit";
        case GC_K_FUSED: return "compress_fused";
        case GC_K_SMALL: return "small_tensors";
        case GC_K_DECODE_TILES: return "decode_tiles";
        case GC_K_FOLD_CAND: return "fold_cand";
        case GC_K_CAND_REFINE: return "cand_refine";
        case GC_K_CAND_COMPACT: return "cand_compact";
        default: return "other";
    }
}

int gc_last_counters(gc_plan_t* p, const void* workspace, void* stream, uint32_t counters[3]) {
    if (p == nullptr || workspace == nullptr || counters == nullptr) return GC_E_INVALID;
    if (p->device < 0) return GC_E_UNSUPPORTED;
    if (!on_plan_device(p)) return GC_E_INVALID;
    WsHeader h;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    GC_CUDA(p, cudaMemcpyAsync(&h, workspace, sizeof(WsHeader), cudaMemcpyDeviceToHost, s));
    GC_CUDA(p, cudaStreamSynchronize(s));
    counters[0] = h.cand_total; counters[1] = h.overflow; counters[2] = h.n_failed;
    return GC_OK;
}

int gc_last_phase_times(gc_plan_t* p, const void* workspace, void* stream, uint64_t ns[20], uint32_t* n_phases) {
    if (p == nullptr || workspace == nullptr || ns == nullptr || n_phases == nullptr) return GC_E_INVALID;
    if (p->device < 0) return GC_E_UNSUPPORTED;
    if (!on_plan_device(p)) return GC_E_INVALID;
    WsHeader h;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    GC_CUDA(p, cudaMemcpyAsync(&h, workspace, sizeof(WsHeader), cudaMemcpyDeviceToHost, s));
    GC_CUDA(p, cudaStreamSynchronize(s));
    uint32_t n = h.n_stamps > 20u ? 20u : h.n_stamps;
    *n_phases = n > 0 ? n - 1 : 0;
    for (uint32_t i = 0; i + 1 < n; ++i) ns[i] = h.stamp[i + 1] - h.stamp[i];
    if (n > 0 && n < 20 && h.t_last_exit > h.stamp[n - 1]) {       // tail: last CTA out after CTA 0's last stamp
        ns[n - 1] = h.t_last_exit - h.stamp[n - 1];
        *n_phases = n;
    }
    return GC_OK;
}

int gc_last_cuda_error(const gc_plan_t* p) { return p ? p->last_cuda_error : 0; }

int gc_destroy(gc_plan_t* p) {
    if (p == nullptr) return GC_OK;
    int rc = GC_OK;
    int caller_device = -1;
    if (p->device >= 0) {                           // the device memory is freed with the plan's device current;
        if (cudaGetDevice(&caller_device) != cudaSuccess) { (void)cudaGetLastError(); caller_device = -1; }
        (void)cudaSetDevice(p->device);             // the caller's device is put back below
    }
    for (auto& r : p->recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    for (auto& u : p->staging) cudaEventDestroy(u.done);
    if (p->ev_copied) cudaEventDestroy(p->ev_copied);
    if (p->copy_stream) cudaStreamDestroy(p->copy_stream);
    if (p->d_small) (void)cudaFree(p->d_small);
    if (p->d_dectile) (void)cudaFree(p->d_dectile);
    if (p->d_desc && cudaFree(p->d_desc) != cudaSuccess) { (void)cudaGetLastError(); rc = GC_E_CUDA; }
    if (caller_device >= 0) (void)cudaSetDevice(caller_device);
    delete p;
    return rc;
}

}  // extern "C"
