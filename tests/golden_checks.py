"""Checks of a result dict (see runners.py) against the hand-worked fixtures
under tests/golden/.  Used for the oracle (CPU) and for the CUDA library."""
import numpy as np

from helpers import bins_of, ints, kv, load_golden


def _device_lane(r):
    d = np.nonzero(r["lane_domain"] == 1)[0]
    assert len(d) == 1
    return int(d[0])


def check_H1(run):
    g = load_golden("H1_gaps.txt")
    r = run(g["events"], [0, len(g["events"])], [g["t0"]], [g["t1"]], min_gap=g["min_gap"])
    e = g["expect"]
    assert r["gap_before"].tolist() == ints(e["gap_before"])
    l = _device_lane(r)
    lg = r["lane_gaps"][l]
    assert lg["busy"] == int(e["lane_busy"][0]) and lg["idle"] == int(e["lane_idle"][0])
    assert lg["busy"] + lg["idle"] == g["t1"] - g["t0"]
    assert lg["n_gaps"] == int(e["lane_n_gaps"][0]) and lg["max_gap"] == int(e["lane_max_gap"][0])
    assert lg["first_start"] == int(e["lane_first_start"][0])
    assert lg["last_end"] == int(e["lane_last_end"][0]) and lg["n_events"] == 6
    hist = np.zeros(40, dtype=np.int64)
    for t in e["hist_bins"]:
        hist += bins_of(t)
    assert r["lane_hist"][l].tolist() == hist.tolist()
    assert r["win_hist"][0].tolist() == hist.tolist()
    want = [tuple(int(x) for x in t.split(",")) for t in e["long_gaps"]]
    got = [(int(x["next_event"]), int(x["gap_start"]), int(x["gap_len"])) for x in r["long_gaps"]]
    assert got == want
    assert all(int(x["lane"]) == l for x in r["long_gaps"])


def check_H2(run):
    g = load_golden("H2_join_attribution.txt")
    n = len(g["events"])
    r = run(g["events"], [0, n], [g["t0"]], [g["t1"]], agg_masks=(1 << 3,))
    e = g["expect"]
    assert r["perm"].tolist() == list(range(n))
    for k in ("parent", "depth", "launch_of", "launch_latency", "queue_delay", "kernels_of_launch",
              "op_of"):
        assert r[k].tolist() == ints(e[k]), k
    for k, v in kv(e["join"]).items():
        assert int(r["join_sum"][0][k]) == v, k
    for k, v in kv(e["attr"]).items():
        assert int(r["attr_sum"][0][k]) == v, k
    assert r["attr_status"] == 0
    seen = set()
    for t in e["op"]:
        pos, rest = t.split(":")
        pos = int(pos)
        nk, first, last, kns = (int(x) for x in rest.split(","))
        assert (int(r["op_n_kernels"][pos]), int(r["op_first_start"][pos]),
                int(r["op_last_end"][pos]), int(r["op_kernel_ns"][pos])) == (nk, first, last, kns)
        seen.add(pos)
    for p in range(n):
        if p not in seen:
            assert r["op_n_kernels"][p] == 0 and r["op_first_start"][p] == 0
            assert r["op_last_end"][p] == 0 and r["op_kernel_ns"][p] == 0
    for pref, key in (("agg0_", "agg_kernel"), ("aggT_", "agg_top")):
        rows = e[key]
        assert len(r[pref + "g_name"]) == len(rows)
        for i, t in enumerate(rows):
            name, rest = t.split(":", 1)
            cnt, sm, mn, mx, bins = rest.split(",", 4)
            assert int(r[pref + "g_window"][i]) == 0 and int(r[pref + "g_pid"][i]) == 1
            assert int(r[pref + "g_name"][i]) == int(name)
            assert (int(r[pref + "g_count"][i]), int(r[pref + "g_sum"][i]),
                    int(r[pref + "g_min"][i]), int(r[pref + "g_max"][i])) == \
                (int(cnt), int(sm), int(mn), int(mx))
            assert r[pref + "g_hist"][i].tolist() == bins_of(bins).tolist()


def check_H3(run):
    g = load_golden("H3_collectives.txt")
    n = len(g["events"])
    r = run(g["events"], [0, n], [g["t0"]], [g["t1"]], comm_sizes=g["comm_sizes"])
    e = g["expect"]
    assert r["c_seq"].tolist() == [0, 1, 2] and r["c_comm"].tolist() == [5, 5, 5]
    for i, t in enumerate(e["groups"]):
        nm, mn, mx, sk, me, st, fl = (int(x) for x in t.split(","))
        got = (int(r["c_n_members"][i]), int(r["c_min_start"][i]), int(r["c_max_start"][i]),
               int(r["c_skew"][i]), int(r["c_max_end"][i]), int(r["c_straggler_pid"][i]),
               int(r["c_flags"][i]))
        assert got == (nm, mn, mx, sk, me, st, fl), i
    waits = {}
    for p in range(n):
        waits[(int(r["pid"][p]), int(r["seq"][p]))] = int(r["wait_ns"][p])
    for t in e["waits"]:
        k, v = t.split(":")
        assert waits[tuple(int(x) for x in k.split(","))] == int(v), t
    assert r["r_pid"].tolist() == [0, 1, 2, 3]
    for t in e["ranks"]:
        pid, rest = t.split(":")
        i = int(pid)
        assert (int(r["r_n_coll"][i]), int(r["r_sum_wait"][i]), int(r["r_max_wait"][i]),
                int(r["r_n_straggler"][i])) == tuple(int(x) for x in rest.split(","))


def check_H4(run):
    g = load_golden("H4_idle_figure.txt")
    n = len(g["events"])
    r = run(g["events"], [0, n], [g["t0"]], [g["t1"]])
    e = g["expect"]
    lg = r["lane_gaps"][0]
    assert lg["busy"] == int(e["lane_busy"][0]) and lg["idle"] == int(e["lane_idle"][0])
    assert lg["n_gaps"] == int(e["lane_n_gaps"][0]) and lg["max_gap"] == int(e["lane_max_gap"][0])
    assert r["gap_before"].sum() == 0
    assert len(r["long_gaps"]) == 1 and r["long_gaps"][0]["next_event"] == -1


def check_H5(run):
    g = load_golden("H5_ties.txt")
    n = len(g["events"])
    r = run(g["events"], [0, n], [g["t0"]], [g["t1"]])
    e = g["expect"]
    assert r["perm"].tolist() == ints(e["perm"])
    assert r["parent"].tolist() == ints(e["parent"])
    assert r["depth"].tolist() == ints(e["depth"])
    assert r["attr_status"] == 0


def check_H6(run):
    g = load_golden("H6_overlap.txt")
    r = run(g["events"], [0, len(g["events"])], [g["t0"]], [g["t1"]])
    want = [tuple(int(x) for x in t.split(":")) for t in g["expect"]["overlap_rows"]]
    got = list(zip(*(r[k].tolist() for k in ("d_pid", "d_n_events", "d_busy", "d_idle", "d_compute",
                                            "d_comm", "d_overlap", "d_exposed"))))
    assert got == want
    assert r["d_window"].tolist() == [0] * len(want)


def check_H7(run):
    g = load_golden("H7_gap_blame.txt")
    r = run(g["events"], [0, len(g["events"])], [g["t0"]], [g["t1"]], min_gap=g["min_gap"])
    e = g["expect"]
    assert r["b_class"].tolist() == ints(e["classes"])
    want = [tuple(int(x) for x in t.split(":")) for t in e["class_totals"]]
    assert [(int(c), int(n)) for c, n in zip(r["b_win_count"][0], r["b_win_ns"][0])] == want
    charged = [tuple(int(x) for x in t.split(":")) for t in e["charged"]]
    got = list(zip(r["aggG_g_name"].tolist(), r["aggG_g_count"].tolist(), r["aggG_g_sum"].tolist()))
    assert got == charged and r["aggG_g_pid"].tolist() == [1, 1]
    assert int(r["op_gap_ns"].sum()) == sum(c[2] for c in charged)


def check_H8(run):
    g = load_golden("H8_rollup.txt")
    r = run(g["events"], [0, len(g["events"])], [g["t0"]], [g["t1"]])
    e = g["expect"]
    assert r["attr_status"] == 0
    for key, name in (("incl_n_kernels", "incl_n"), ("incl_kernel_ns", "incl_ns"),
                      ("incl_first_start", "incl_first"), ("incl_last_end", "incl_last"),
                      ("replay_first_start", "replay_first"), ("replay_last_end", "replay_last"),
                      ("replay_kernel_ns", "replay_ns")):
        assert r[key].tolist() == ints(e[name]), key
    assert r["roll_sum"][0].tolist() == ints(e["roll_sum"])


def check_H9(run):
    g = load_golden("H9_critical_path.txt")
    r = run(g["events"], [0, len(g["events"])], [g["t0"]], [g["t1"]])
    e = g["expect"]
    assert r["cp_window"].tolist() == [0, 0] and r["cp_pid"].tolist() == ints(e["pids"])
    assert r["cp_begin"].tolist() == ints(e["begin"]) and r["cp_end"].tolist() == ints(e["end"])
    assert r["cp_reason"].tolist() == ints(e["reason"]) and r["cp_n_nodes"].tolist() == ints(e["n_nodes"])
    want = [[int(x) for x in t.split(":")] for t in e["ns"]]
    assert r["cp_ns"].reshape(-1, 8).tolist() == want
    on = np.nonzero(r["on_path"])[0]
    assert r["ts_start"][on].tolist() == ints(e["on_path"])
    assert r["ts_start"][r["cp_sink"]].tolist() == ints(e["sinks"])
    assert r["cp_sum"].reshape(-1, 10)[0].tolist() == [2, 10] + [a + b for a, b in zip(*want)]
    sym = [tuple(int(x) for x in t.split(":")) for t in e["on_path_symbols"]]
    assert list(zip(r["aggP_g_pid"].tolist(), r["aggP_g_name"].tolist(), r["aggP_g_count"].tolist(),
                    r["aggP_g_sum"].tolist())) == sym


def check_H10(run):
    g = load_golden("H10_depth_boundary.txt")
    ev = g["events"]
    n = len(ev)
    r = run(ev, [0, n], [g["t0"]], [g["t1"]])
    e = g["expect"]
    assert r["perm"].tolist() == list(range(n))
    assert r["parent"].tolist() == ints(e["parent"])
    assert r["depth"].tolist() == ints(e["depth"])
    assert r["op_of"].tolist() == ints(e["op_of"])
    assert r["attr_status"] == 0
    for k, v in kv(e["attr"]).items():
        assert int(r["attr_sum"][0][k]) == v, k
    # the fixture's encloser counts, from the enclosure rule itself (records are in canonical
    # order, one host lane); the surplus over the depth = enclosers that are no ancestors
    want_enc = ints(e["enclosers"])
    for i in range(n):
        if ev[i]["kind"] > 2:
            assert want_enc[i] == 0
            continue
        enc = [j for j in range(n) if j != i and ev[j]["kind"] == 0
               and ev[j]["ts_start"] <= ev[i]["ts_start"] and ev[i]["ts_end"] <= ev[j]["ts_end"]
               and ((ev[j]["ts_start"], ev[j]["ts_end"]) != (ev[i]["ts_start"], ev[i]["ts_end"]) or j < i)]
        assert len(enc) == want_enc[i], i
        chain, c = [], int(r["parent"][i])
        while c >= 0:
            chain.append(c)
            c = int(r["parent"][c])
        assert set(chain) <= set(enc)
        assert want_enc[i] - int(r["depth"][i]) == len(set(enc) - set(chain)), i


def check_H11(run):
    g = load_golden("H11_operator_sol.txt")
    n = len(g["events"])
    r = run(g["events"], [0, n], [g["t0"]], [g["t1"]], op_work=g["op_work"])
    e = g["expect"]
    assert r["perm"].tolist() == list(range(n)) and r["attr_status"] == 0
    assert r["sol_state"].tolist() == ints(e["sol_state"])
    for k in ("sol_mfu", "sol_mbu", "sol_op"):
        want = np.array([float(t) for t in e[k]])
        # T_op * 1e-9 s is rounded (1e-9 is no binary fraction): a few units in the last place
        assert np.allclose(r[k], want, rtol=1e-12, atol=0), k
        assert np.array_equal(r[k] == 0, want == 0), k
    s = r["sol_sum"][0]
    for t in e["sol_sum"]:
        k, v = t.split("=")
        assert abs(float(s[k]) - float(v)) <= 1e-12 * abs(float(v)), k


ALL = [check_H1, check_H2, check_H3, check_H4, check_H5, check_H6, check_H7, check_H8, check_H9, check_H10, check_H11]
