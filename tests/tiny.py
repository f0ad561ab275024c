"""Random tiny adversarial windows for brute-force and parity tests."""
import numpy as np

from helpers import make_events


def _nested(rng, a, b, depth, max_depth, rows, pid, tid, n_names, corr_pool, p_launch=0.5):
    """Fills [a, b] with properly nested OP ranges and launches; many ties."""
    t = a
    while t <= b and rng.random() < 0.85:
        if rng.random() < p_launch or depth >= max_depth:
            e = min(b, t + int(rng.integers(0, 4)))
            kind = "LAUNCH" if rng.random() < 0.8 else "API"
            corr = int(rng.choice(corr_pool))
            rows.append((kind, pid, tid, t, e, corr, int(rng.integers(0, n_names)), 0))
            t = e + int(rng.integers(0, 3))
        else:
            e = min(b, t + int(rng.integers(0, max(1, (b - t) // 2 + 1))))
            rows.append(("OP", pid, tid, t, e, 0, int(rng.integers(0, n_names)), 0))
            _nested(rng, t, e, depth + 1, max_depth, rows, pid, tid, n_names, corr_pool, p_launch)
            t = e + int(rng.integers(0, 3))


def random_window(seed, span=400, n_pid=3, n_dev=60, max_depth=5, n_names=5, defects=True,
                  nested=True, n_windows=2, colls=True):
    """Returns (events, win_off, t0, t1, comm_sizes).  Small time range so that equal
    timestamps, zero-length records and identical intervals are common."""
    rng = np.random.default_rng(seed)
    all_rows = []
    win_off = [0]
    t0s, t1s = [], []
    pids = [-7, 3, 100000][:n_pid]
    corr_pool = [0, 1, 2, 3, 5, -1, 2**40 + 1, 7, 8, 9, 10, 11]
    for w in range(n_windows):
        t0 = int(10**6 * (w + 1) + rng.integers(0, 50))
        t1 = t0 + span
        rows = []
        for pid in pids:
            for tid in range(int(rng.integers(1, 3))):
                if nested:
                    _nested(rng, t0, t1 - 1, 0, max_depth, rows, pid, tid, n_names, corr_pool)
                else:
                    for _ in range(int(rng.integers(3, 12))):
                        s = int(rng.integers(t0, t1))
                        e = s + int(rng.integers(0, 40))
                        kind = ["OP", "OP", "LAUNCH", "API"][int(rng.integers(0, 4))]
                        rows.append((kind, pid, tid, s, e, int(rng.choice(corr_pool)),
                                     int(rng.integers(0, n_names)), 0))
            for _ in range(n_dev // n_pid):
                s = int(rng.integers(t0, t1))
                e = s + int(rng.integers(0, 30)) if rng.random() < 0.9 else t1 + int(rng.integers(0, 50))
                kind = ["KERNEL", "KERNEL", "MEMCPY"][int(rng.integers(0, 3))]
                rows.append((kind, pid, int(rng.integers(0, 3)) - 1, s, e, int(rng.choice(corr_pool)),
                             int(rng.integers(0, n_names)), 0))
            if colls:
                for sq in range(4):
                    if rng.random() < 0.85:
                        s = int(rng.integers(t0, t1))
                        rows.append(("COLL", pid, 1, s, s + int(rng.integers(0, 20)),
                                     int(rng.choice([5, -3])), 0, sq))
                    if rng.random() < 0.1:  # duplicate pid inside a group
                        s = int(rng.integers(t0, t1))
                        rows.append(("COLL", pid, 0, s, s + 3, 5, 0, sq))
        if defects:
            for _ in range(4):
                s = int(rng.integers(t0, t1))
                which = int(rng.integers(0, 4))
                pid = pids[int(rng.integers(0, len(pids)))]
                if which == 0:
                    rows.append((int(rng.choice([-1, 6, 77])), pid, 0, s, s + 1, 0, 0, 0))
                elif which == 1:
                    rows.append(("KERNEL", pid, 0, s, s - 1 - int(rng.integers(0, 5)), 0, 0, 0))
                elif which == 2:
                    rows.append(("OP", pid, 0, t0 - 1 - int(rng.integers(0, 5)), s, 0, 0, 0))
                else:
                    rows.append(("LAUNCH", pid, 0, t1 + int(rng.integers(0, 5)), t1 + 9, 1, 0, 0))
        order = rng.permutation(len(rows))
        rows = [rows[i] for i in order]
        all_rows += rows
        win_off.append(len(all_rows))
        t0s.append(t0)
        t1s.append(t1)
    return make_events(all_rows), win_off, t0s, t1s, [(5, n_pid)]


def schedule_window(seed, tight=False, n_actions=40, n_streams=3, n_pid=2):
    """A simulated run per process: one host thread issues launches and waits, every stream runs
    its kernels in order.  tight=True: a kernel starts exactly when its launch call starts or
    the stream frees up, whichever is later, and a wait returns a fixed time after the last
    kernel ends; otherwise random latencies and some records without a launch are mixed in.
    Returns (events, win_off, t0, t1, info) with info[pid] = dict(first, makespan, dag)."""
    rng = np.random.default_rng(1000 + seed)
    rows, info = [], {}
    corr = 1
    for pid in range(1, n_pid + 1):
        t = int(rng.integers(5, 50))
        first = None
        free = [0] * n_streams
        last_host_end = None
        edges = []  # (from point, to point, weight) of the full dependency graph, tight mode
        prev_dev = [None] * n_streams
        devs = []
        for _ in range(n_actions):
            if rng.random() < 0.75:
                s = int(rng.integers(0, n_streams))
                a = int(rng.integers(1, 8))
                dur = int(rng.integers(1, 60))
                lat = 0 if tight else int(rng.integers(0, 12))
                me = ("L", corr)
                rows.append(("LAUNCH", pid, 0, t, t + a, corr, 0, 0))
                start = max(t + lat, free[s])
                if tight or rng.random() < 0.9:
                    kind = "KERNEL" if rng.random() < 0.8 else "MEMCPY"
                    rows.append((kind, pid, s, start, start + dur, corr, 0, 0))
                    k = ("K", corr)
                    edges.append((("S", me), ("S", k), 0))
                    if prev_dev[s] is not None:
                        edges.append((("E", prev_dev[s]), ("S", k), 0))
                    edges.append((("S", k), ("E", k), dur))
                    prev_dev[s] = k
                    devs.append(k)
                    free[s] = start + dur
                elif rng.random() < 0.5:  # a device record whose launch was not captured
                    rows.append(("KERNEL", pid, s, start, start + dur, 10_000 + corr, 0, 0))
                    free[s] = start + dur
                corr += 1
                end = t + a
            else:
                me = ("A", corr)
                tail = int(rng.integers(1, 6))
                end = max(t, max(free)) + tail if (tight or rng.random() < 0.8) else t + tail
                rows.append(("API", pid, 0, t, end, 0, 0, 0))
                for k in devs:
                    edges.append((("E", k), ("E", me), tail))
                edges.append((("S", me), ("E", me), tail))
                corr += 1
            if me[0] == "L":
                edges.append((("S", me), ("E", me), end - t))
            if last_host_end is not None:
                edges.append((("E", last_host_end[0]), ("S", me), t - last_host_end[1]))
            else:
                first = (me, t)
            last_host_end = (me, end)
            t = end + int(rng.integers(0, 15))
        if not tight and rng.random() < 0.5:
            rows.append(("COLL", pid, n_streams, int(rng.integers(0, 40)), int(rng.integers(40, 90)), 5, 0, 0))
        info[pid] = dict(first=first[1], makespan=max(max(free), last_host_end[1]) - first[1],
                         edges=edges, source=("S", first[0]))
    order = rng.permutation(len(rows))
    ev = make_events([rows[i] for i in order])
    hi = int(max(r[4] for r in rows)) + 10
    return ev, [0, len(ev)], [0], [hi], info
