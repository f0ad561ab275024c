"""Shared test helpers: golden-fixture parser and small record builders."""
import os

import numpy as np

from paper_2609_40247_b200.synth import EVENT_DTYPE

KINDS = {"OP": 0, "API": 1, "LAUNCH": 2, "KERNEL": 3, "MEMCPY": 4, "COLL": 5}
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def make_events(rows):
    """rows: iterable of (kind, pid, stream, s, e, corr, name, seq)."""
    rows = list(rows)
    ev = np.zeros(len(rows), dtype=EVENT_DTYPE)
    for i, (kind, pid, stream, s, e, corr, name, seq) in enumerate(rows):
        ev[i] = (s, e, corr, pid, name, seq, stream, KINDS[kind] if isinstance(kind, str) else kind)
    return ev


def load_golden(name):
    """Parses tests/golden/<name>: returns dict(events, t0, t1, min_gap, comm_sizes, expect
    [, op_work = (flops, bytes, peak_flops, peak_bw)])."""
    rows, expect, comm, work = [], {}, [], []
    t0 = t1 = None
    peaks = None
    min_gap = 1
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            tok = line.split()
            if tok[0] == "window":
                t0, t1 = int(tok[1]), int(tok[2])
            elif tok[0] == "event":
                rows.append((tok[1], int(tok[2]), int(tok[3]), int(tok[4]), int(tok[5]),
                             int(tok[6]), int(tok[7]), int(tok[8])))
            elif tok[0] == "repeat_kernels":
                cnt, dur = int(tok[1]), int(tok[2])
                for i in range(cnt):
                    rows.append(("KERNEL", 1, 0, t0 + i * dur, t0 + (i + 1) * dur, 0, 0, 0))
            elif tok[0] == "min_gap":
                min_gap = int(tok[1])
            elif tok[0] == "peaks":
                peaks = (float(tok[1]), float(tok[2]))
            elif tok[0] == "work":
                work.append((int(tok[1]), float(tok[2]), float(tok[3])))
            elif tok[0] == "comm_size":
                comm.append((int(tok[1]), int(tok[2])))
            elif tok[0] == "expect":
                expect[tok[1]] = tok[2:]
            else:
                raise ValueError(line)
    g = dict(events=make_events(rows), t0=t0, t1=t1, min_gap=min_gap, comm_sizes=comm,
             expect=expect)
    if peaks is not None:  # per input record: operation count and data volume, -1 = not known
        flops = np.full(len(rows), -1.0)
        nbytes = np.full(len(rows), -1.0)
        for k, f, b in work:
            flops[k], nbytes[k] = f, b
        g["op_work"] = (flops, nbytes, peaks[0], peaks[1])
    return g


def ints(tokens):
    return [int(t) for t in tokens]


def kv(tokens):
    return {t.split("=")[0]: int(t.split("=")[1]) for t in tokens}


def bins_of(spec):
    """'4:1;5:2' -> 40-vector."""
    h = np.zeros(40, dtype=np.int64)
    for part in spec.split(";"):
        b, c = part.split(":")
        h[int(b)] = int(c)
    return h
