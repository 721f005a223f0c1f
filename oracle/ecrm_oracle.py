"""CPU oracle of the erasure-coded embedding-table path.  TEST INFRASTRUCTURE ONLY: nothing in
the product may import this module (tests, the smoke check and the benchmark's CPU-baseline
legs do).

Plain numpy, float32 throughout, one rounded operation at a time, sums in the order written:
what Sections 3.2-3.4 of the source define (encoder p = e_1 + ... + e_k, decoder
e_i = p - sum of the others, the optimizer step of Section 3.3.1 for Adagrad, server-side
propagation of the DIFFERENCES of entry and optimizer state, degraded reads, rotating parity
placement).  Readings where the source is silent are marked "reading" below.
"""
from __future__ import annotations

import numpy as np

ADAGRAD, MOMENTUM = 0, 1
f32 = np.float32


def encode(shards):
    """Summation encoder, Section 3.2: p = ((e_1 + e_2) + e_3) + ... (reading: left to right)."""
    p = np.array(shards[0], dtype=f32, copy=True)
    for s in shards[1:]:
        p = (p + np.asarray(s, dtype=f32)).astype(f32)
    return p


def decode(parity, survivors):
    """Subtraction decoder, Section 3.2: e_i = ((p - e_a) - e_b) - ... over the k-1 survivors in
    the order given (reading: left to right)."""
    out = np.array(parity, dtype=f32, copy=True)
    for s in survivors:
        out = (out - np.asarray(s, dtype=f32)).astype(f32)
    return out


def rows_step(optimizer, rows, grad, entry, state, lr, hyper):
    """Optimizer applied to the rows of a batch (in place) + the differences that server-side
    propagation sends (Section 3.3.2).  Adagrad as written in Section 3.3.1:
    G' = G + g^2, e' = e - (lr / sqrt(G' + eps)) g.  Momentum SGD (the evaluation's optimizer,
    formula not printed; reading: v' = mu v + g, e' = e - lr v').
    Returns (d_entry, d_state) with d = fl(new - old), row j of the batch at position j."""
    lr, hyper = f32(lr), f32(hyper)
    grad = np.asarray(grad, dtype=f32)
    d_entry = np.empty_like(grad)
    d_state = np.empty_like(grad)
    for j, row in enumerate(np.asarray(rows)):
        g, e, s = grad[j], entry[row].copy(), state[row].copy()
        if optimizer == ADAGRAD:
            sn = (s + (g * g).astype(f32)).astype(f32)
            step = (lr / np.sqrt((sn + hyper).astype(f32)).astype(f32)).astype(f32)
            en = (e - (step * g).astype(f32)).astype(f32)
        elif optimizer == MOMENTUM:
            sn = ((hyper * s).astype(f32) + g).astype(f32)
            en = (e - (lr * sn).astype(f32)).astype(f32)
        else:
            raise ValueError(optimizer)
        d_entry[j] = (en - e).astype(f32)
        d_state[j] = (sn - s).astype(f32)
        entry[row], state[row] = en, sn
    return d_entry, d_state


def parity_add(prow, d_entry, d_state, p_entry, p_state):
    """The parity host adds the received differences (Section 3.3.2), in place."""
    for j, row in enumerate(np.asarray(prow)):
        p_entry[row] = (p_entry[row] + d_entry[j]).astype(f32)
        if p_state is not None:
            p_state[row] = (p_state[row] + d_state[j]).astype(f32)


def degraded_read(prow, srows, shards, parity):
    """Rows of the failed server from the parity row and the k-1 surviving rows (Section 3.4)."""
    prow = np.asarray(prow)
    out = np.array(parity[prow], dtype=f32, copy=True)
    for s, shard in enumerate(shards):
        r = prow if srows is None or srows[s] is None else np.asarray(srows[s])
        out = (out - shard[r]).astype(f32)
    return out


def placement(k, group):
    """Rotating parity placement over k+1 servers (Section 3.2, after RAID-5): the parity of
    group number `group` lives on server group mod (k+1), its k entries on the others in
    increasing server number (reading: the figure shows the rotation, not a formula)."""
    ps = int(group) % (k + 1)
    return ps, [s for s in range(k + 1) if s != ps]
