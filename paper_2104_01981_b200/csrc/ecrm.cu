// Erasure-coded embedding-table hot path: summation encoder / subtraction decoder over whole
// shards, the optimizer step that emits entry and state differences, the parity host's
// scatter-add of those differences, and degraded reads.  Everything is bound by HBM traffic:
// rows are 512-byte (dim = 128) contiguous runs, one warp moves one row with 128-bit accesses.
#include <cuda_runtime.h>
#include <stdint.h>

#include "ecrm.h"

namespace {

constexpr int kThreads = 256;
constexpr int kWarpsPerCta = kThreads / 32;

struct PtrTable { const float* p[ECRM_MAX_K]; };
struct RowTable { const uint32_t* p[ECRM_MAX_K]; };

// out = first (+|-) p[0] (+|-) p[1] ... elementwise in that order; SUB selects the decoder.
// `first` is nullptr for the encoder (the sum then starts from p[0]).
template <bool SUB>
__global__ void __launch_bounds__(kThreads) k_ecrm_combine(PtrTable t, uint32_t k, const float* first,
                                                            float* out, uint64_t n) {   // out may be first
    const uint64_t n4 = n / 4;
    const uint64_t stride = (uint64_t)gridDim.x * kThreads;
    for (uint64_t i = (uint64_t)blockIdx.x * kThreads + threadIdx.x; i < n4; i += stride) {
        float4 acc;
        uint32_t s = 0;
        if (SUB) acc = __ldcs(reinterpret_cast<const float4*>(first) + i);
        else { acc = __ldcs(reinterpret_cast<const float4*>(t.p[0]) + i); s = 1; }
        for (; s + 4 <= k; s += 4) {                    // four shard loads in flight
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = __ldcs(reinterpret_cast<const float4*>(t.p[s + u]) + i);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (SUB) { acc.x = __fsub_rn(acc.x, v[u].x); acc.y = __fsub_rn(acc.y, v[u].y);
                           acc.z = __fsub_rn(acc.z, v[u].z); acc.w = __fsub_rn(acc.w, v[u].w); }
                else     { acc.x = __fadd_rn(acc.x, v[u].x); acc.y = __fadd_rn(acc.y, v[u].y);
                           acc.z = __fadd_rn(acc.z, v[u].z); acc.w = __fadd_rn(acc.w, v[u].w); }
            }
        }
        for (; s < k; ++s) {
            const float4 v = __ldcs(reinterpret_cast<const float4*>(t.p[s]) + i);
            if (SUB) { acc.x = __fsub_rn(acc.x, v.x); acc.y = __fsub_rn(acc.y, v.y);
                       acc.z = __fsub_rn(acc.z, v.z); acc.w = __fsub_rn(acc.w, v.w); }
            else     { acc.x = __fadd_rn(acc.x, v.x); acc.y = __fadd_rn(acc.y, v.y);
                       acc.z = __fadd_rn(acc.z, v.z); acc.w = __fadd_rn(acc.w, v.w); }
        }
        __stcs(reinterpret_cast<float4*>(out) + i, acc);
    }
    // ragged tail (n not a multiple of 4)
    for (uint64_t i = n4 * 4 + (uint64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += stride) {
        float acc;
        uint32_t s = 0;
        if (SUB) acc = first[i]; else { acc = t.p[0][i]; s = 1; }
        for (; s < k; ++s) acc = SUB ? __fsub_rn(acc, t.p[s][i]) : __fadd_rn(acc, t.p[s][i]);
        out[i] = acc;
    }
}

// One warp per updated row.  OPT: ECRM_ADAGRAD or ECRM_MOMENTUM.
template <int OPT>
__global__ void __launch_bounds__(kThreads) k_ecrm_rows_step(uint32_t m, const uint32_t* __restrict__ rows,
                                                              const float* __restrict__ grad, float* __restrict__ entry,
                                                              float* __restrict__ state, uint64_t n_rows, uint32_t dim4,
                                                              float lr, float hyper, float* __restrict__ d_entry,
                                                              float* __restrict__ d_state, uint32_t* bad_rows) {
    const int lane = threadIdx.x & 31;
    const uint64_t warp = (uint64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    const uint64_t nwarps = (uint64_t)gridDim.x * kWarpsPerCta;
    for (uint64_t j = warp; j < m; j += nwarps) {
        const uint32_t row = __ldg(rows + j);
        if (row >= n_rows) {
            if (lane == 0 && bad_rows != nullptr) atomicAdd(bad_rows, 1u);
            continue;
        }
        const float4* g4 = reinterpret_cast<const float4*>(grad) + j * dim4;
        float4* e4 = reinterpret_cast<float4*>(entry) + (uint64_t)row * dim4;
        float4* s4 = reinterpret_cast<float4*>(state) + (uint64_t)row * dim4;
        float4* de4 = reinterpret_cast<float4*>(d_entry) + j * dim4;
        float4* ds4 = reinterpret_cast<float4*>(d_state) + j * dim4;
        for (uint32_t c = lane; c < dim4; c += 32) {
            const float4 g = __ldcs(g4 + c);
            const float4 e = e4[c];
            const float4 s = s4[c];
            const float gv[4] = {g.x, g.y, g.z, g.w}, ev[4] = {e.x, e.y, e.z, e.w}, sv[4] = {s.x, s.y, s.z, s.w};
            float en[4], sn[4], de[4], ds[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (OPT == ECRM_ADAGRAD) {
                    sn[q] = __fadd_rn(sv[q], __fmul_rn(gv[q], gv[q]));
                    const float step = __fdiv_rn(lr, __fsqrt_rn(__fadd_rn(sn[q], hyper)));
                    en[q] = __fsub_rn(ev[q], __fmul_rn(step, gv[q]));
                } else {
                    sn[q] = __fadd_rn(__fmul_rn(hyper, sv[q]), gv[q]);
                    en[q] = __fsub_rn(ev[q], __fmul_rn(lr, sn[q]));
                }
                de[q] = __fsub_rn(en[q], ev[q]);
                ds[q] = __fsub_rn(sn[q], sv[q]);
            }
            e4[c] = make_float4(en[0], en[1], en[2], en[3]);
            s4[c] = make_float4(sn[0], sn[1], sn[2], sn[3]);
            __stcs(de4 + c, make_float4(de[0], de[1], de[2], de[3]));
            __stcs(ds4 + c, make_float4(ds[0], ds[1], ds[2], ds[3]));
        }
    }
}

// The optimizer step and the parity update of the same rows in one pass, for a data shard whose
// parity lives on the same GPU: the two differences stay in registers.  One warp per row.
template <int OPT>
__global__ void __launch_bounds__(kThreads) k_ecrm_rows_step_parity(uint32_t m, const uint32_t* __restrict__ rows,
                                                                     const uint32_t* __restrict__ prow,
                                                                     const float* __restrict__ grad, float* __restrict__ entry,
                                                                     float* __restrict__ state, uint64_t n_rows,
                                                                     float* __restrict__ p_entry, float* __restrict__ p_state,
                                                                     uint64_t n_prows, uint32_t dim4, float lr, float hyper,
                                                                     uint32_t* bad_rows) {
    const int lane = threadIdx.x & 31;
    const uint64_t warp = (uint64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    const uint64_t nwarps = (uint64_t)gridDim.x * kWarpsPerCta;
    for (uint64_t j = warp; j < m; j += nwarps) {
        const uint32_t row = __ldg(rows + j), pr = __ldg(prow + j);
        if (row >= n_rows || pr >= n_prows) {
            if (lane == 0 && bad_rows != nullptr) atomicAdd(bad_rows, 1u);
            continue;
        }
        const float4* g4 = reinterpret_cast<const float4*>(grad) + j * dim4;
        float4* e4 = reinterpret_cast<float4*>(entry) + (uint64_t)row * dim4;
        float4* s4 = reinterpret_cast<float4*>(state) + (uint64_t)row * dim4;
        float4* pe4 = reinterpret_cast<float4*>(p_entry) + (uint64_t)pr * dim4;
        float4* ps4 = reinterpret_cast<float4*>(p_state) + (uint64_t)pr * dim4;
        for (uint32_t c = lane; c < dim4; c += 32) {
            const float4 g = __ldcs(g4 + c);
            const float4 e = e4[c], s = s4[c], pe = pe4[c], ps = ps4[c];
            const float gv[4] = {g.x, g.y, g.z, g.w}, ev[4] = {e.x, e.y, e.z, e.w}, sv[4] = {s.x, s.y, s.z, s.w};
            const float pev[4] = {pe.x, pe.y, pe.z, pe.w}, psv[4] = {ps.x, ps.y, ps.z, ps.w};
            float en[4], sn[4], pen[4], psn[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (OPT == ECRM_ADAGRAD) {
                    sn[q] = __fadd_rn(sv[q], __fmul_rn(gv[q], gv[q]));
                    const float step = __fdiv_rn(lr, __fsqrt_rn(__fadd_rn(sn[q], hyper)));
                    en[q] = __fsub_rn(ev[q], __fmul_rn(step, gv[q]));
                } else {
                    sn[q] = __fadd_rn(__fmul_rn(hyper, sv[q]), gv[q]);
                    en[q] = __fsub_rn(ev[q], __fmul_rn(lr, sn[q]));
                }
                pen[q] = __fadd_rn(pev[q], __fsub_rn(en[q], ev[q]));      // parity += fl(new - old), as the two calls do
                psn[q] = __fadd_rn(psv[q], __fsub_rn(sn[q], sv[q]));
            }
            e4[c] = make_float4(en[0], en[1], en[2], en[3]);
            s4[c] = make_float4(sn[0], sn[1], sn[2], sn[3]);
            pe4[c] = make_float4(pen[0], pen[1], pen[2], pen[3]);
            ps4[c] = make_float4(psn[0], psn[1], psn[2], psn[3]);
        }
    }
}

// One warp per parity row: p += d (entry and, if given, state).
__global__ void __launch_bounds__(kThreads) k_ecrm_parity_add(uint32_t m, const uint32_t* __restrict__ prow,
                                                               const float* __restrict__ d_entry,
                                                               const float* __restrict__ d_state,
                                                               float* __restrict__ p_entry, float* __restrict__ p_state,
                                                               uint64_t n_prows, uint32_t dim4, uint32_t* bad_rows) {
    const int lane = threadIdx.x & 31;
    const uint64_t warp = (uint64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    const uint64_t nwarps = (uint64_t)gridDim.x * kWarpsPerCta;
    for (uint64_t j = warp; j < m; j += nwarps) {
        const uint32_t row = __ldg(prow + j);
        if (row >= n_prows) {
            if (lane == 0 && bad_rows != nullptr) atomicAdd(bad_rows, 1u);
            continue;
        }
        for (uint32_t c = lane; c < dim4; c += 32) {
            float4* pe = reinterpret_cast<float4*>(p_entry) + (uint64_t)row * dim4 + c;
            const float4 d = __ldcs(reinterpret_cast<const float4*>(d_entry) + j * dim4 + c);
            float4 p = *pe;
            p.x = __fadd_rn(p.x, d.x); p.y = __fadd_rn(p.y, d.y); p.z = __fadd_rn(p.z, d.z); p.w = __fadd_rn(p.w, d.w);
            *pe = p;
            if (p_state != nullptr) {
                float4* ps = reinterpret_cast<float4*>(p_state) + (uint64_t)row * dim4 + c;
                const float4 d2 = __ldcs(reinterpret_cast<const float4*>(d_state) + j * dim4 + c);
                float4 q = *ps;
                q.x = __fadd_rn(q.x, d2.x); q.y = __fadd_rn(q.y, d2.y); q.z = __fadd_rn(q.z, d2.z); q.w = __fadd_rn(q.w, d2.w);
                *ps = q;
            }
        }
    }
}

// One warp per requested row: parity row minus the surviving rows, in shard order.
__global__ void __launch_bounds__(kThreads) k_ecrm_degraded_read(uint32_t k_avail, uint32_t m,
                                                                  const uint32_t* __restrict__ prow, RowTable srow,
                                                                  PtrTable shards, const float* __restrict__ parity,
                                                                  uint64_t n_rows, uint32_t dim4,
                                                                  float* __restrict__ out, uint32_t* bad_rows) {
    const int lane = threadIdx.x & 31;
    const uint64_t warp = (uint64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    const uint64_t nwarps = (uint64_t)gridDim.x * kWarpsPerCta;
    for (uint64_t j = warp; j < m; j += nwarps) {
        const uint32_t pr = __ldg(prow + j);
        bool ok = pr < n_rows;
        uint32_t sr[ECRM_MAX_K];
        for (uint32_t s = 0; s < k_avail; ++s) {
            sr[s] = srow.p[s] != nullptr ? __ldg(srow.p[s] + j) : pr;
            ok = ok && sr[s] < n_rows;
        }
        if (!ok) {
            if (lane == 0 && bad_rows != nullptr) atomicAdd(bad_rows, 1u);
            continue;
        }
        for (uint32_t c = lane; c < dim4; c += 32) {
            float4 acc = reinterpret_cast<const float4*>(parity)[(uint64_t)pr * dim4 + c];
            for (uint32_t s = 0; s < k_avail; ++s) {
                const float4 v = reinterpret_cast<const float4*>(shards.p[s])[(uint64_t)sr[s] * dim4 + c];
                acc.x = __fsub_rn(acc.x, v.x); acc.y = __fsub_rn(acc.y, v.y);
                acc.z = __fsub_rn(acc.z, v.z); acc.w = __fsub_rn(acc.w, v.w);
            }
            __stcs(reinterpret_cast<float4*>(out) + j * dim4 + c, acc);
        }
    }
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int grid_for_rows(uint32_t m) {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) (void)cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const uint64_t want = ((uint64_t)m + kWarpsPerCta - 1) / kWarpsPerCta;
    const uint64_t cap = (uint64_t)sms * 8 * 4;          // a few waves of resident CTAs, then a row loop
    return (int)(want < cap ? (want ? want : 1) : cap);
}

int launched() { return cudaGetLastError() == cudaSuccess ? ECRM_OK : ECRM_E_CUDA; }

}  // namespace

extern "C" {

int ecrm_encode(uint32_t k, const float* const* shards, float* parity, uint64_t n, void* stream) {
    if (k < 1 || k > ECRM_MAX_K || shards == nullptr || parity == nullptr || !aligned16(parity)) return ECRM_E_INVALID;
    PtrTable t{};
    for (uint32_t s = 0; s < k; ++s) {
        if (shards[s] == nullptr || !aligned16(shards[s]) || shards[s] == parity) return ECRM_E_INVALID;
        t.p[s] = shards[s];
    }
    if (n == 0) return ECRM_OK;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) (void)cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const uint64_t want = (n / 4 + kThreads - 1) / kThreads + 1;
    const int grid = (int)(want < (uint64_t)sms * 16 ? want : (uint64_t)sms * 16);
    k_ecrm_combine<false><<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(t, k, nullptr, parity, n);
    return launched();
}

int ecrm_decode(uint32_t k_avail, const float* const* shards, const float* parity, float* out, uint64_t n,
                void* stream) {
    if (k_avail >= ECRM_MAX_K || parity == nullptr || out == nullptr || !aligned16(parity) || !aligned16(out) ||
        (k_avail > 0 && shards == nullptr))
        return ECRM_E_INVALID;
    PtrTable t{};
    for (uint32_t s = 0; s < k_avail; ++s) {
        if (shards[s] == nullptr || !aligned16(shards[s]) || shards[s] == out) return ECRM_E_INVALID;
        t.p[s] = shards[s];
    }
    if (n == 0) return ECRM_OK;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) (void)cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const uint64_t want = (n / 4 + kThreads - 1) / kThreads + 1;
    const int grid = (int)(want < (uint64_t)sms * 16 ? want : (uint64_t)sms * 16);
    k_ecrm_combine<true><<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(t, k_avail, parity, out, n);
    return launched();
}

int ecrm_rows_step(int optimizer, uint32_t m, const uint32_t* rows, const float* grad, float* entry, float* state,
                   uint64_t n_rows, uint32_t dim, float lr, float hyper, float* d_entry, float* d_state,
                   uint32_t* bad_rows, void* stream) {
    if (optimizer != ECRM_ADAGRAD && optimizer != ECRM_MOMENTUM) return ECRM_E_INVALID;
    if (dim == 0 || (dim & 3u) != 0 || n_rows == 0 || n_rows > 0xFFFFFFFFull) return ECRM_E_INVALID;
    if (m == 0) return ECRM_OK;
    if (rows == nullptr || grad == nullptr || entry == nullptr || state == nullptr || d_entry == nullptr ||
        d_state == nullptr)
        return ECRM_E_INVALID;
    if (!aligned16(grad) || !aligned16(entry) || !aligned16(state) || !aligned16(d_entry) || !aligned16(d_state))
        return ECRM_E_INVALID;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int grid = grid_for_rows(m);
    if (optimizer == ECRM_ADAGRAD)
        k_ecrm_rows_step<ECRM_ADAGRAD><<<grid, kThreads, 0, s>>>(m, rows, grad, entry, state, n_rows, dim / 4, lr,
                                                                  hyper, d_entry, d_state, bad_rows);
    else
        k_ecrm_rows_step<ECRM_MOMENTUM><<<grid, kThreads, 0, s>>>(m, rows, grad, entry, state, n_rows, dim / 4, lr,
                                                                   hyper, d_entry, d_state, bad_rows);
    return launched();
}

int ecrm_rows_step_parity(int optimizer, uint32_t m, const uint32_t* rows, const uint32_t* prow, const float* grad,
                          float* entry, float* state, uint64_t n_rows, float* p_entry, float* p_state, uint64_t n_prows,
                          uint32_t dim, float lr, float hyper, uint32_t* bad_rows, void* stream) {
    if (optimizer != ECRM_ADAGRAD && optimizer != ECRM_MOMENTUM) return ECRM_E_INVALID;
    if (dim == 0 || (dim & 3u) != 0 || n_rows == 0 || n_rows > 0xFFFFFFFFull || n_prows == 0 || n_prows > 0xFFFFFFFFull)
        return ECRM_E_INVALID;
    if (m == 0) return ECRM_OK;
    if (rows == nullptr || prow == nullptr || grad == nullptr || entry == nullptr || state == nullptr ||
        p_entry == nullptr || p_state == nullptr)
        return ECRM_E_INVALID;
    if (!aligned16(grad) || !aligned16(entry) || !aligned16(state) || !aligned16(p_entry) || !aligned16(p_state))
        return ECRM_E_INVALID;
    if (p_entry == entry || p_state == state || p_entry == state || p_state == entry) return ECRM_E_INVALID;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int grid = grid_for_rows(m);
    if (optimizer == ECRM_ADAGRAD)
        k_ecrm_rows_step_parity<ECRM_ADAGRAD><<<grid, kThreads, 0, s>>>(m, rows, prow, grad, entry, state, n_rows, p_entry,
                                                                         p_state, n_prows, dim / 4, lr, hyper, bad_rows);
    else
        k_ecrm_rows_step_parity<ECRM_MOMENTUM><<<grid, kThreads, 0, s>>>(m, rows, prow, grad, entry, state, n_rows, p_entry,
                                                                          p_state, n_prows, dim / 4, lr, hyper, bad_rows);
    return launched();
}

int ecrm_parity_add(uint32_t m, const uint32_t* prow, const float* d_entry, const float* d_state, float* p_entry,
                    float* p_state, uint64_t n_prows, uint32_t dim, uint32_t* bad_rows, void* stream) {
    if (dim == 0 || (dim & 3u) != 0 || n_prows == 0 || n_prows > 0xFFFFFFFFull) return ECRM_E_INVALID;
    if (m == 0) return ECRM_OK;
    if (prow == nullptr || d_entry == nullptr || p_entry == nullptr || (d_state == nullptr) != (p_state == nullptr))
        return ECRM_E_INVALID;
    if (!aligned16(d_entry) || !aligned16(p_entry) || !aligned16(d_state) || !aligned16(p_state)) return ECRM_E_INVALID;
    k_ecrm_parity_add<<<grid_for_rows(m), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        m, prow, d_entry, d_state, p_entry, p_state, n_prows, dim / 4, bad_rows);
    return launched();
}

int ecrm_degraded_read(uint32_t k_avail, uint32_t m, const uint32_t* prow, const uint32_t* const* srow,
                       const float* const* shards, const float* parity, uint64_t n_rows, uint32_t dim, float* out,
                       uint32_t* bad_rows, void* stream) {
    if (k_avail >= ECRM_MAX_K || dim == 0 || (dim & 3u) != 0 || n_rows == 0 || n_rows > 0xFFFFFFFFull)
        return ECRM_E_INVALID;
    if (m == 0) return ECRM_OK;
    if (prow == nullptr || parity == nullptr || out == nullptr || (k_avail > 0 && shards == nullptr) ||
        !aligned16(parity) || !aligned16(out))
        return ECRM_E_INVALID;
    PtrTable t{};
    RowTable rt{};
    for (uint32_t s = 0; s < k_avail; ++s) {
        if (shards[s] == nullptr || !aligned16(shards[s])) return ECRM_E_INVALID;
        t.p[s] = shards[s];
        rt.p[s] = srow != nullptr ? srow[s] : nullptr;
    }
    k_ecrm_degraded_read<<<grid_for_rows(m), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        k_avail, m, prow, rt, t, parity, n_rows, dim / 4, out, bad_rows);
    return launched();
}

int ecrm_placement(uint32_t k, uint64_t group, uint32_t* parity_server, uint32_t* data_servers) {
    if (k < 1 || k > ECRM_MAX_K || parity_server == nullptr || data_servers == nullptr) return ECRM_E_INVALID;
    const uint32_t ps = (uint32_t)(group % (uint64_t)(k + 1));
    *parity_server = ps;
    uint32_t j = 0;
    for (uint32_t s = 0; s <= k; ++s)
        if (s != ps) data_servers[j++] = s;
    return ECRM_OK;
}

}  // extern "C"
