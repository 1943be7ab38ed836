"""Label-level prediction of the selection on the prototype workloads.

On the synthetic generator two tokens are strongly correlated (|cos| >= ~0.97)
exactly when they currently carry the same prototype label, and nearly
orthogonal (|cos| <~ 0.2) otherwise.  With thr = 0.91 "correlated" therefore
means "same label", and Definition 1 / Algorithm 1 can be replayed on the
labels alone -- no norms, no Gram -- which gives an independent prediction of
the index sets at any size.  Unique tokens carry distinct negative labels.
"""
import numpy as np


def full_from_labels(labels):
    """Definition 1 on labels: t is representative iff no earlier token shares its label."""
    seen = set()
    rep = []
    for t, lab in enumerate(labels.tolist()):
        if lab not in seen:
            rep.append(t)
            seen.add(lab)
    return np.asarray(rep, dtype=np.int32)


def cascade_from_labels(labels, rep_in, causal=False):
    """Algorithm 1 on labels.  Returns (rep_out, add, rem)."""
    labels = labels.tolist()
    rep_in = [int(x) for x in rep_in]
    in_set = set(rep_in)
    seen = set()
    valid, rem = [], []
    for s in rep_in:                      # lines 3-5: against ALL earlier inherited reps
        if labels[s] in seen:
            rem.append(s)
        else:
            valid.append(s)
        seen.add(labels[s])
    first_valid_pos = {}
    for s in valid:
        first_valid_pos.setdefault(labels[s], s)
    add = []
    for t in range(len(labels)):          # lines 6-9
        if t in in_set:
            continue
        s = first_valid_pos.get(labels[t])
        covered = s is not None and (not causal or s < t)
        if not covered:
            add.append(t)
    rep_out = sorted(valid + add)
    return (np.asarray(rep_out, dtype=np.int32), np.asarray(add, dtype=np.int32),
            np.asarray(rem, dtype=np.int32))
