/*
 * ecrm.h -- C ABI of the erasure-coded embedding-table hot path (same library, libgc.so).
 *
 * What it covers: the server-side work of erasure-coded recommendation-model training with one
 * parity per k embedding-table entries (r = 1):
 *   - summation encoder   p = e_1 + e_2 + ... + e_k and subtraction decoder
 *     e_i = p - sum of the other k-1 entries            (Section 3.2, "Encoder and decoder")
 *   - the optimizer applied to the rows a batch touched, which also emits the DIFFERENCES of
 *     entry and optimizer state, and the parity host adding those differences to the parity
 *     entry and the parity optimizer state              (Section 3.3.2, server-side propagation)
 *   - reading a row of a failed server from the k-1 surviving rows and the parity
 *     ("degraded read", Section 3.4), and full recovery of a shard (the same decoder over
 *     whole arrays)
 *   - rotating parity placement over k+1 servers        (Section 3.2, "Where should parities
 *     be placed?")
 * Locks and buffering during recovery, the network and the training system around it are not
 * here.
 *
 * Layout: an embedding table shard is a dense fp32 matrix [n_rows][dim], row-major, dim a
 * multiple of 4 (the evaluated model uses dim = 128, Section 4.1); optimizer state has the same
 * shape (one float of state per parameter).  All data pointers are DEVICE pointers owned by
 * the caller, 16-byte aligned.  Pointer tables (`shards`) are HOST arrays of device pointers.
 * Every call is asynchronous on `stream` (cudaStream_t, 0 = legacy default) and allocates
 * nothing.
 *
 * Arithmetic: fp32, every operation rounded once (no fused multiply-add), sums taken in the
 * order written below, so results are bit-reproducible.  A decoded entry equals the lost one
 * exactly when all partial sums are exactly representable (e.g. integer-valued data) and to
 * within (k+1) roundings of the parity's magnitude otherwise: the code is a floating-point
 * sum, as in the source; it is not a bit-level (XOR) code.
 *
 * Return value: ECRM_OK (0) or a negative error: ECRM_E_INVALID (null pointer, bad size,
 * misaligned pointer, k out of range), ECRM_E_CUDA (launch failed; see gc_last_cuda_error-like
 * detail via cudaGetLastError by the caller).  Row indices that are out of range are skipped
 * and counted in *bad_rows when that pointer (device, may be NULL) is given.
 */
#ifndef ECRM_H
#define ECRM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ECRM_OK          0
#define ECRM_E_INVALID  (-1)
#define ECRM_E_CUDA     (-3)

#define ECRM_MAX_K      32

/* optimizers of ecrm_rows_step */
#define ECRM_ADAGRAD    0   /* state' = state + g*g;  entry' = entry - (lr / sqrt(state' + hyper)) * g,
                               hyper = epsilon                       (the update written out in Section 3.3.1) */
#define ECRM_MOMENTUM   1   /* state' = hyper * state + g;  entry' = entry - lr * state',  hyper = momentum
                               (SGD with momentum, the optimizer of the evaluation, Section 4.1; the source
                               does not print its formula -- this is the accumulate-then-step form) */

/*
 * ecrm_encode -- parity[i] = ((shards[0][i] + shards[1][i]) + shards[2][i]) + ... for i < n.
 *   k        1..ECRM_MAX_K data shards of n floats each; parity: n floats, may not alias a shard.
 */
int ecrm_encode(uint32_t k, const float *const *shards, float *parity, uint64_t n, void *stream);

/*
 * ecrm_decode -- out[i] = ((parity[i] - shards[0][i]) - shards[1][i]) - ... for i < n: the lost
 * shard from the parity and the k_avail = k-1 surviving shards (0..ECRM_MAX_K-1 of them), in the
 * order given.  out may alias parity (recovering in place) but no shard.
 */
int ecrm_decode(uint32_t k_avail, const float *const *shards, const float *parity, float *out,
                uint64_t n, void *stream);

/*
 * ecrm_rows_step -- applies the optimizer to the m rows a batch touched and emits the
 * differences that server-side propagation sends to the parity host.
 *   rows      device, uint32[m]: row numbers, each at most once (a batch's gradient is already
 *             aggregated per row); any order
 *   grad      device, fp32[m][dim]: gradient of row rows[j] at position j
 *   entry, state  device, fp32[n_rows][dim]: updated in place
 *   d_entry, d_state  device, fp32[m][dim]: fl(entry' - entry) and fl(state' - state), position j
 *   lr, hyper see ECRM_ADAGRAD / ECRM_MOMENTUM
 */
int ecrm_rows_step(int optimizer, uint32_t m, const uint32_t *rows, const float *grad,
                   float *entry, float *state, uint64_t n_rows, uint32_t dim, float lr, float hyper,
                   float *d_entry, float *d_state, uint32_t *bad_rows, void *stream);

/*
 * ecrm_parity_add -- the parity host's side: p_entry[prow[j]] += d_entry[j] and
 * p_state[prow[j]] += d_state[j] (one rounded add per element).  prow: device, uint32[m], each
 * parity row at most once per call (differences for the same parity row coming from different
 * data servers arrive in different calls, and calls on one stream apply in order).
 * p_state / d_state may both be NULL (optimizer without state).
 */
int ecrm_parity_add(uint32_t m, const uint32_t *prow, const float *d_entry, const float *d_state,
                    float *p_entry, float *p_state, uint64_t n_prows, uint32_t dim,
                    uint32_t *bad_rows, void *stream);

/*
 * ecrm_rows_step_parity -- ecrm_rows_step and ecrm_parity_add of the same rows in one pass, for a
 * data shard whose parity shard lives on the same GPU (Section 3.3.2: the differences that
 * server-side propagation would send never leave the chip, so they are not written out).
 * For every j < m: the optimizer step on row rows[j] of entry / state exactly as in
 * ecrm_rows_step, then p_entry[prow[j]] += fl(entry' - entry) and p_state[prow[j]] +=
 * fl(state' - state), one rounding per operation -- bit for bit what the two calls give.
 *   rows, prow   device, uint32[m]; every data row and every parity row at most once per call
 *   the parity arrays must not be the data arrays; a row number out of range (either table)
 *   skips the row and is counted in *bad_rows
 * Moves 9 rows of dim floats per updated row instead of 13.
 */
int ecrm_rows_step_parity(int optimizer, uint32_t m, const uint32_t *rows, const uint32_t *prow, const float *grad,
                          float *entry, float *state, uint64_t n_rows, float *p_entry, float *p_state,
                          uint64_t n_prows, uint32_t dim, float lr, float hyper, uint32_t *bad_rows, void *stream);

/*
 * ecrm_degraded_read -- out[j] = ((parity[prow[j]] - shards[0][srow[0][j]]) - shards[1][srow[1][j]]) ...
 * for j < m: rows of the failed server rebuilt on the fly.
 *   prow      device, uint32[m]: parity row of request j
 *   srow      HOST array of k_avail DEVICE pointers, uint32[m] each: the row of surviving shard s
 *             that belongs to the same group; NULL entry = same row number as prow
 *   out       device, fp32[m][dim]
 */
int ecrm_degraded_read(uint32_t k_avail, uint32_t m, const uint32_t *prow, const uint32_t *const *srow,
                       const float *const *shards, const float *parity, uint64_t n_rows, uint32_t dim,
                       float *out, uint32_t *bad_rows, void *stream);

/*
 * ecrm_placement -- host only.  Rotating parity placement over k+1 servers: group number
 * `group` keeps its parity on server group mod (k+1), and its k entries on the other servers
 * in increasing server number: data_servers[0..k-1].  Every server ends up with the same
 * number of parities.
 */
int ecrm_placement(uint32_t k, uint64_t group, uint32_t *parity_server, uint32_t *data_servers);

#ifdef __cplusplus
}
#endif
#endif /* ECRM_H */
