// Threshold-estimation variant: after the exact k_s-th largest key tau of each tensor's sample
// is known, ONE pass folds the residual, sends every element with key >= tau in index order
// (at most `cap` per tensor) and zeroes what it sent: 12 bytes per element plus 8 per hit.
#pragma once
#include "gc_kernels.cuh"

namespace gc {

// Ticket-ordered tiles; the number of hits before a tile (within its tensor) comes from the
// look-back exchange, so output slots are index-ordered and a truncated tensor keeps exactly
// its first `cap` hits.  tau of tensor t = ssel[t].T, or `tau_fixed` when ssel is null.
// FOLD: a = g + r is computed here (and stored); otherwise r already holds a.
// SKIP_SMALL: tensors of kind "small" were finished elsewhere and are left alone.
template <bool FOLD, bool SKIP_SMALL = false>
static __device__ void threshold_emit_body(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles,
                                           const float* __restrict__ g, float* __restrict__ r,
                                           uint32_t* __restrict__ out_idx, float* __restrict__ out_val,
                                           uint32_t* __restrict__ out_count, const WsView& ws,
                                           const TensorSel* __restrict__ ssel, uint32_t tau_fixed, int ticket_slot) {
    __shared__ uint32_t s_tile;
    __shared__ uint32_t s_tot[kWarps], s_ex[kWarps];
    __shared__ uint32_t s_sum;
    __shared__ unsigned long long s_excl;
    __shared__ int s_ok;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    while (true) {
        __syncthreads();
        if (tid == 0) {
            uint32_t tk = atomicAdd(&ws.hdr->ticket[ticket_slot], 1u);
            if (*(volatile uint32_t*)&ws.hdr->abort) tk = 0xFFFFFFFFu;
            s_tile = tk;
        }
        __syncthreads();
        const uint32_t tile = s_tile;
        if (tile >= ntiles) break;
        const uint32_t t = find_tensor(desc, T, tile);
        const TensorDesc d = desc[t];
        if (SKIP_SMALL && d.kind == kKindSmall) continue;
        const uint32_t tau = ssel != nullptr ? ssel[t].T : tau_fixed;
        const TileGeom tg = tile_geom(d, tile - d.tile0);
        Tile tl;
        load_tile<FOLD>(g, r, tg, warp, lane, tl);

        uint32_t cnt[kVpt], hm = 0;
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
            cnt[j] = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                bool h = ((tl.valid >> (4 * j + e)) & 1u) && key_of(tl.a[j][e]) >= tau;
                cnt[j] += h;
                hm |= (uint32_t)h << (4 * j + e);
            }
        }
        uint32_t rk[kVpt], wtot;
        warp_rank(cnt, lane, rk, wtot);
        if (lane == 0) s_tot[warp] = wtot;
        __syncthreads();
        scan_warp_totals(s_tot, s_ex, &s_sum, warp, lane);
        __syncthreads();
        if (warp == 0) {
            bool ok;
            unsigned long long ex = lookback(ws.tile_state, tile, d.tile0, (unsigned long long)s_sum, lane,
                                             ws.hdr, ok);
            if (lane == 0) { s_excl = ex; s_ok = ok ? 1 : 0; }
        }
        __syncthreads();
        if (!s_ok) break;
        const uint32_t before = (uint32_t)s_excl + s_ex[warp];
        if (hm != 0u) {
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                uint32_t slot = before + rk[j];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if ((hm >> (4 * j + e)) & 1u) {
                        if (slot < d.cap) {
                            uint32_t f = vec_index(tg.base, warp, lane, j) + e;
                            out_idx[d.out_off + slot] = f;
                            out_val[d.out_off + slot] = tl.a[j][e];
                            r[f] = 0.0f;
                        }
                        ++slot;
                    }
                }
            }
        }
        if (tile == d.tile0 + d.ntiles - 1 && tid == 0) {
            const uint32_t hits = (uint32_t)s_excl + s_sum;
            if (out_count != nullptr) {
                out_count[t] = min(hits, d.cap);
                out_count[T + t] = hits;
            }
            if (hits > d.cap) record_status(ws.hdr, 1 /*GC_W_TRUNCATED*/, t);
        }
    }
}

static __global__ void __launch_bounds__(kBlock)
k_threshold_emit(const TensorDesc* __restrict__ desc, uint32_t T, uint32_t ntiles,
                 const float* __restrict__ g, float* __restrict__ r,
                 uint32_t* __restrict__ out_idx, float* __restrict__ out_val,
                 uint32_t* __restrict__ out_count, WsView ws, const TensorSel* __restrict__ ssel,
                 int ticket_slot) {
    threshold_emit_body<true>(desc, T, ntiles, g, r, out_idx, out_val, out_count, ws, ssel, 0u, ticket_slot);
}

}  // namespace gc
