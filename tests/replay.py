"""Per-ID replay: a second, independent statement of the table's rules.

Under the batch semantics of the table every ID's state depends only on its
own history -- the steps it occurred in, its multiplicity and summed gradient
in each, and the sweep schedule -- never on other IDs (as long as the row
capacity is not exhausted).  This module replays one ID at a time through a
small state machine written in numpy scalars.  It knows nothing about bags of
other IDs, maps or ordering, so it fails differently from the map-based oracle
when either is wrong.
"""
from __future__ import annotations

import numpy as np

f32 = np.float32


def id_histories(steps):
    """steps: list of (ids, offsets, grad, now, sweep: bool).

    Returns {id: [(step_index, multiplicity, summed_grad_f64), ...]}.
    """
    hist = {}
    for si, (ids, offsets, grad, now, sweep) in enumerate(steps):
        bag_of = np.repeat(np.arange(offsets.size - 1), np.diff(offsets))
        per = {}
        for j, id_ in enumerate(ids.tolist()):
            if id_ == 0xFFFFFFFFFFFFFFFF:
                continue
            m, g = per.get(id_, (0, np.zeros(grad.shape[1], np.float64)))
            per[id_] = (m + 1, g + grad[bag_of[j]].astype(np.float64))
        for id_, (m, g) in per.items():
            hist.setdefault(id_, []).append((si, m, g))
    return hist


def replay_id(id_, events, steps, *, threshold, ttl, lr, eps, init_acc, init_row):
    """Final state of one ID.  init_row(id) -> float32 vector of initial values."""
    T = max(threshold, 1)
    tracked, count, seen, resident = False, 0, -1, False
    w = acc = None
    ev = {si: (m, g) for si, m, g in events}
    for si, (_, _, _, now, sweep) in enumerate(steps):
        if si in ev:
            m, g = ev[si]
            if not tracked:
                tracked, count, resident = True, 0, False
            count = min(count + m, T)
            seen = now
            if not resident and count >= T:
                resident = True
                w = init_row(id_).astype(f32).copy()
                acc = np.full_like(w, f32(init_acc))
            if resident:
                G = g.astype(f32)
                acc = (acc + G * G).astype(f32)
                w = (w - f32(lr) * G / (np.sqrt(acc).astype(f32) + f32(eps))).astype(f32)
        if sweep and tracked and ttl > 0 and now - seen > ttl:
            tracked, count, resident, w, acc = False, 0, False, None, None
    return {"tracked": tracked, "count": count if tracked else 0,
            "last_seen": seen if tracked else -1, "resident": resident, "w": w, "acc": acc}
