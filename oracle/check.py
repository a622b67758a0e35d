"""Acceptance rule that compares a retrieval result with the oracle's scores.

Test infrastructure only.  The rule is the one the task states for this path:
every returned score within `tol` of the oracle's score for that entry, and the
returned id set equal to the oracle's top-k except where oracle scores tie
within `tol` around the k-th place.  Nothing here computes a similarity; the
oracle's full score matrix is an input.
"""
from __future__ import annotations

import numpy as np


class AcceptanceError(AssertionError):
    pass


def accept(got_ids, got_scores, all_scores, k: int, ids=None, tol: float = 2e-2,
           what: str = "") -> dict:
    """Check got_ids/got_scores [nq,k] against oracle scores all_scores [nq,n].

    ids: the int64 labels the cache rows were inserted with (default: slot).
    Labels must be unique so that a returned id names one row.
    Returns a small report (max |score error|, number of boundary-ambiguous
    entries); raises AcceptanceError on the first violated rule.
    """
    got_ids = np.asarray(got_ids)
    got_scores = np.asarray(got_scores, dtype=np.float32)
    all_scores = np.asarray(all_scores, dtype=np.float32)
    nq, n = all_scores.shape
    if got_ids.shape != (nq, k) or got_scores.shape != (nq, k):
        raise AcceptanceError(f"{what}: result shape {got_ids.shape}/{got_scores.shape}, expected {(nq, k)}")
    if ids is None:
        slot_of = None
    else:
        ids = np.asarray(ids, dtype=np.int64)
        sorter = np.argsort(ids, kind="stable")
        sorted_ids = ids[sorter]
        if n > 1 and np.any(sorted_ids[1:] == sorted_ids[:-1]):
            raise ValueError("labels must be unique for the acceptance check")
    real = min(k, n)
    max_err = 0.0
    ambiguous = 0
    for iq in range(nq):
        gi, gs = got_ids[iq], got_scores[iq]
        # Rule 1: count, padding, uniqueness, order.
        if np.any(gi[real:] != -1) or not np.all(np.isneginf(gs[real:])):
            raise AcceptanceError(f"{what} q{iq}: tail past min(k,n) is not (-1, -inf)")
        if real == 0:
            continue
        gi_r, gs_r = gi[:real], gs[:real]
        if ids is None:
            slots = gi_r.astype(np.int64)
            if np.any(slots < 0) or np.any(slots >= n):
                raise AcceptanceError(f"{what} q{iq}: returned id outside the cache")
        else:
            pos = np.searchsorted(sorted_ids, gi_r)
            pos = np.clip(pos, 0, n - 1)
            if np.any(sorted_ids[pos] != gi_r):
                raise AcceptanceError(f"{what} q{iq}: returned id that was never inserted")
            slots = sorter[pos]
        if np.unique(slots).size != real:
            raise AcceptanceError(f"{what} q{iq}: an entry is returned twice")
        if np.any(np.isnan(gs_r)) or np.any(gs_r[1:] > gs_r[:-1]):
            raise AcceptanceError(f"{what} q{iq}: scores are not sorted descending")
        # Rule 2: score accuracy.
        o = all_scores[iq]
        err = np.abs(gs_r.astype(np.float64) - o[slots].astype(np.float64))
        worst = float(err.max())
        max_err = max(max_err, worst)
        if worst > tol:
            j = int(err.argmax())
            raise AcceptanceError(
                f"{what} q{iq}: score {gs_r[j]!r} for id {gi_r[j]} differs from oracle "
                f"{o[slots[j]]!r} by {worst:.3e} > {tol:.1e}")
        # Rule 3: id set, modulo ties within tol around the k-th oracle score.
        if real < n:
            t_k = np.partition(o, n - real)[n - real]
        else:
            t_k = o.min()
        low = o[slots] < t_k - tol
        if np.any(low):
            j = int(np.argmax(low))
            raise AcceptanceError(
                f"{what} q{iq}: id {gi_r[j]} (oracle {o[slots[j]]!r}) is below the k-th oracle "
                f"score {t_k!r} by more than {tol:.1e}")
        must = np.flatnonzero(o > t_k + tol)
        missing = np.setdiff1d(must, slots, assume_unique=False)
        if missing.size:
            raise AcceptanceError(
                f"{what} q{iq}: slot {int(missing[0])} (oracle {o[missing[0]]!r}) beats the k-th "
                f"oracle score {t_k!r} by more than {tol:.1e} but was not returned")
        ambiguous += int(np.count_nonzero(np.abs(o - t_k) <= tol))
    return {"max_abs_err": max_err, "boundary_entries": ambiguous, "queries": nq}
