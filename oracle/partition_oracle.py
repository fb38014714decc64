"""Algorithm 1 (partitioning for balanced pipeline generation), plain Python.

TEST INFRASTRUCTURE ONLY (see the package docstring).

Inputs are per-layer costs: ``T_fix[l]`` (immovable work: forward + G) and
``T_flex[l]`` (movable work: the delta computation of layer l, which may be
borrowed by the processor holding layer l+1), and the processor target N_p.
The layers are walked in reverse; processors are filled one after another up
to the per-processor budget ``T_p = T_tot / N_p``; a delta that does not fit is
split by operational parallelism into delta'' (fills what is left of the
current processor) and delta' (goes to the next one).  If more processors than
N_p are needed the budget is relaxed by a factor alpha and step 3 restarts.

Readings of the printed algorithm (the box is garbled or silent at these
points; each is repeated in the design notes):
  * T_tot is the sum over layers of T_fix + T_flex; all arithmetic is integer,
    T_p = ceil(T_tot / N_p), alpha = 101/100 applied as ceil(T_p * 101 / 100).
  * When the fixed part does not fit and the processor index advances, the
    idle time restarts from T_p before T_fix is subtracted (otherwise the
    worked example of Table III cannot be reproduced).
  * Processors used = p_idx + 1; relax iff that exceeds N_p; fewer than N_p is
    accepted.
  * OP(T_idle, T_flex): delta'' = max(0, T_idle), delta' = T_flex - delta''.
    A layer with T_flex = 0 has nothing to place and is skipped.
  * Comparisons are strict as printed: flex fits iff T_flex < T_idle; fix
    advances iff T_fix > T_idle.
  * Reverse processor index p (0 = last pipeline stage) maps to stage
    ``used - 1 - p``.  Layer l's forward, G and update live where T_fix[l] was
    placed, and d_l = used - 1 - stage(l) is its delay (one per stage after it).
"""


def partition(T_fix, T_flex, n_proc, alpha_num=101, alpha_den=100, max_rounds=100000):
    L = len(T_fix)
    T_fix = [int(t) for t in T_fix]
    T_flex = [int(t) for t in T_flex]
    T_tot = sum(T_fix) + sum(T_flex)
    T_p = -(-T_tot // n_proc)
    rounds = 0
    while True:
        p_idx, T_idle = 0, T_p
        fix_proc = [0] * L
        pieces = [[] for _ in range(L)]          # per layer: [(reverse proc, amount, tag)]
        for l in reversed(range(L)):
            if T_flex[l] > 0:
                if T_flex[l] < T_idle:
                    pieces[l].append((p_idx, T_flex[l], "whole"))
                    T_idle -= T_flex[l]
                else:
                    d2 = max(0, T_idle)
                    d1 = T_flex[l] - d2
                    pieces[l].append((p_idx, d2, "delta''"))
                    p_idx += 1
                    pieces[l].append((p_idx, d1, "delta'"))
                    T_idle = T_p - d1
            if T_fix[l] > T_idle:
                p_idx += 1
                T_idle = T_p
            fix_proc[l] = p_idx
            T_idle -= T_fix[l]
        used = p_idx + 1
        if used > n_proc:
            T_p = -(-T_p * alpha_num // alpha_den)
            rounds += 1
            if rounds > max_rounds:
                raise RuntimeError("relaxation did not terminate")
        else:
            break
    stage = [used - 1 - p for p in fix_proc]
    delay = [used - 1 - s for s in stage]
    dgrad = [[(used - 1 - p, amt, tag) for (p, amt, tag) in pl] for pl in pieces]
    loads = [0] * used
    for l in range(L):
        loads[stage[l]] += T_fix[l]
        for (s, amt, _) in dgrad[l]:
            loads[s] += amt
    return dict(stage=stage, delay=delay, dgrad=dgrad, used=used, T_p=T_p,
                relax_rounds=rounds, loads=loads)


def layer_granular_partition(T_total, n_proc):
    """The comparison baseline of Table III: whole layers (backward as one task)
    in contiguous groups, minimising the largest group (exhaustive search; only
    for small examples)."""
    from itertools import combinations
    L = len(T_total)
    best = None
    for cuts in combinations(range(1, L), n_proc - 1):
        edges = (0,) + cuts + (L,)
        loads = [sum(T_total[edges[i]:edges[i + 1]]) for i in range(n_proc)]
        if best is None or max(loads) < max(best[1]):
            best = (edges, loads)
    return best


def mac_costs(layers, batch):
    """Integer cost model used in place of a profiler: multiply-accumulates of
    the true shapes.  fix = forward + G = 2 x MACs, flex = delta = MACs, and the
    first layer needs no delta (nothing consumes dE/da^0)."""
    fix, flex = [], []
    for i, l in enumerate(layers):
        if l["kind"] == "fc":
            macs = batch * l["n_in"] * l["n_out"]
        else:
            Ho = (l["H"] + 2 * l["pad"] - l["R"]) // l["stride"] + 1
            Wo = (l["W"] + 2 * l["pad"] - l["S"]) // l["stride"] + 1
            macs = batch * Ho * Wo * l["n_out"] * l["R"] * l["S"] * l["n_in"]
        fix.append(2 * macs)
        flex.append(macs if i > 0 else 0)
    return fix, flex
