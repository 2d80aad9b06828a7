"""Pins the oracle's Algorithm 2 to trajectories worked by hand from the paper's text.

tests/golden/alg2_handworked.txt holds four tiny instances with the level vector after every
iteration, each derived on paper from Algorithm 2's lines (Section 4.2).  Both oracle forms
must walk them: the whole-loop allocator and a host loop over the single-iteration step
(acceptance decided here from the table, as the caller of the step would).
"""
import os

import numpy as np
import pytest

from oracle import sbo

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "alg2_handworked.txt")


def _load():
    cases, cur, mode = [], None, None
    for raw in open(GOLDEN):
        line = raw.split("#", 1)[0].strip()
        if not line:
            continue
        tok = line.split()
        if tok[0] == "instance":
            cur = {"name": tok[1], "table": [], "trace": []}
            cases.append(cur)
            mode = None
        elif tok[0] in ("bits", "block_elems"):
            cur[tok[0]] = [int(t) for t in tok[1:]]
        elif tok[0] in ("budget", "gamma0", "gammaT"):
            cur[tok[0]] = float(tok[1])
        elif tok[0] in ("table", "trace"):
            mode = tok[0]
        elif tok[0] == "final":
            cur["final"] = {tok[i]: float(tok[i + 1]) for i in range(1, len(tok), 2)}
            mode = None
        elif mode == "table":
            cur["table"].append([float(t) for t in tok])
        elif mode == "trace":
            cur["trace"].append([int(t) for t in tok])
        else:
            raise ValueError(f"cannot parse: {raw!r}")
    return cases


CASES = _load()


def test_the_file_holds_the_cases_the_step_rules_need():
    assert len(CASES) >= 4
    for c in CASES:
        N, L = len(c["table"]), len(c["bits"])
        assert all(len(r) == L for r in c["table"]) and len(c["block_elems"]) == N
        assert all(len(t) == N for t in c["trace"])
        assert len(c["trace"]) == int(c["final"]["iterations"])
        # the file's own bookkeeping: budget and loss of the last vector
        last = c["trace"][-1]
        used = sum(m * c["bits"][l] for m, l in zip(c["block_elems"], last))
        assert used == int(c["final"]["used_bits"]) <= int(c["final"]["cap_bits"])
        assert sum(c["table"][i][l] for i, l in enumerate(last)) == c["final"]["loss_final"]
        assert int(np.floor(c["budget"] * sum(c["block_elems"]))) == int(c["final"]["cap_bits"])


@pytest.mark.parametrize("case", CASES, ids=[c["name"] for c in CASES])
def test_whole_loop_allocator_walks_the_handworked_trajectory(case):
    E = np.array(case["table"], dtype=np.float64)
    sizes = np.array(case["block_elems"], dtype=np.int64)
    st, level, rep, trace = sbo.allocate_scalebits_trace(
        E, case["bits"], case["budget"], case["gamma0"], case["gammaT"], 0, block_elems=sizes)
    assert st == sbo.OK
    want = np.array(case["trace"], dtype=np.uint8)
    assert trace.shape == want.shape, (trace, want)
    for t in range(want.shape[0]):
        assert np.array_equal(trace[t], want[t]), f"iteration {t + 1}: {trace[t]} != {want[t]}"
    assert np.array_equal(level, want[-1])
    fin = case["final"]
    for key in ("iterations", "expansions", "accepted", "rejected", "used_bits", "cap_bits"):
        assert rep[key] == int(fin[key]), key
    assert rep["proxy_loss_init"] == fin["loss_init"]
    assert rep["proxy_loss_final"] == fin["loss_final"]
    # the plain entry point returns the same allocation
    st2, level2, rep2 = sbo.allocate_scalebits(E, case["bits"], case["budget"], case["gamma0"],
                                               case["gammaT"], 0, block_elems=sizes)
    assert st2 == sbo.OK and np.array_equal(level2, level) and rep2["iterations"] == rep["iterations"]


@pytest.mark.parametrize("case", CASES, ids=[c["name"] for c in CASES])
def test_single_iteration_step_walks_the_handworked_trajectory(case):
    E = np.array(case["table"], dtype=np.float64)
    sizes = np.array(case["block_elems"], dtype=np.int64)
    bits, budget = case["bits"], case["budget"]
    N, L = E.shape
    idx = np.arange(N)
    level = np.full(N, max(l for l in range(L) if bits[l] <= budget), dtype=np.uint8)
    k = max(1, int(np.floor(case["gamma0"] * N)))
    kT = max(1, int(np.floor(case["gammaT"] * N)))
    k = max(k, kT)
    got, counts = [], {"expansions": 0, "accepted": 0, "rejected": 0}
    while k >= kT:
        assert len(got) < 64
        lv = level.astype(np.int64)
        s_up = np.where(lv + 1 < L, E[idx, lv] - E[idx, np.minimum(lv + 1, L - 1)], 0.0)
        s_dn = np.where(lv > 0, E[idx, np.maximum(lv - 1, 0)] - E[idx, lv], 0.0)
        st, out, rep = sbo.exchange_step(s_up, s_dn, level, bits, budget, k, 0, block_elems=sizes)
        assert st == sbo.OK
        loss_now, loss_new = E[idx, lv].sum(), E[idx, out.astype(np.int64)].sum()
        if rep["moved"] and rep["expansion"]:
            level = out
            counts["expansions"] += 1
        elif rep["moved"] and loss_new < loss_now:       # line 11: keep unless the loss rose
            level = out
            counts["accepted"] += 1
        else:
            k //= 2                                       # line 12
            counts["rejected"] += 1
        got.append(level.copy())
    want = np.array(case["trace"], dtype=np.uint8)
    assert len(got) == want.shape[0]
    for t in range(want.shape[0]):
        assert np.array_equal(got[t], want[t]), f"iteration {t + 1}: {got[t]} != {want[t]}"
    for key, v in counts.items():
        assert v == int(case["final"][key]), key
