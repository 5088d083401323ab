"""Planner oracle: checkpoint-selection objectives written out as plain definitions.

TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct CPU statement of what the
host planner and the activation arena must reproduce.  It shares no code with the library under
``paper_2502_12499_b200/`` and must never be imported by it; only ``tests/``, the smoke check and
the benchmark's CPU-baseline leg call it.  Objectives, simulators and enumeration are exact Python integers; the static recursion holds
its tables in numpy int64 (guarded against overflow) so that n = 1000 finishes in seconds.

Notation follows the paper: sizes ``d[0..n]`` (``d[0]`` = input, ``d[n]`` = output), a checkpoint
set ``C`` that always contains 0 and n (Section 3.1), segments = the non-checkpoints between two
consecutive checkpoints.

Functions and the passage each one restates:

* ``eval_static``      - Eq. (cost): sum of checkpoints + the largest segment sum.
* ``eval_dynamic``     - Eq. (memory)/(memory-simple) with s(h,i) of Eq. (s): max over checkpoints i
                         of [checkpoints up to i + segment before i + largest d_k, h <= k < i].
* ``simulate_alg1``    - Algorithm 1 (store everything) as an allocation event list.
* ``simulate_alg2``    - Algorithm 2 (batch free) as an allocation event list.
* ``simulate_alg4``    - Algorithm 4 (early free + one output-gradient buffer per segment) as an
                         allocation event list.  Reading taken where the listing and Eq. (memory)
                         disagree: the previous gradient buffer is released *before* the segment is
                         recomputed, so that the event high-water equals Eq. (memory) exactly.
* ``stage_trace``      - bytes at the end of every training phase index of Section 5.1.1.
* ``brute_force_static`` / ``brute_force_dynamic`` - the optimum by enumerating every feasible set
                         (2^(n-1) of the 2^n masks over d_1..d_n contain n), plus the canonical
                         optimal set under the tie rule stated below.
* ``dp_static_reference``  - Eq. (T) per segment cap, scanned directly (no queue), caps = all
                         contiguous range sums of d_1..d_{n-1} plus 0, output d_n forced.
* ``dp_dynamic_reference`` - Algorithm 5 (the O(n^2) recursion of Eq. (T-rec)) with i running down
                         to 0 and j up to n inclusive.
* ``eval_two_size`` / ``brute_force_two_size`` / ``dp_two_size_reference`` - Eq. (memory) with three sizes per
                         tensor instead of one (the more faithful allocator model the paper's Section 6 leaves as
                         future work, following Observations (1)-(2) of Section 4): what d_t occupies as a
                         checkpoint, what it occupies inside the segment being processed, and the size of its
                         gradient; optionally with the buffer of the *incoming* gradient counted next to the
                         paper's output-gradient buffer.  With all three sizes equal to d and no incoming buffer
                         it is Eq. (memory) itself.

Tie rule (the paper gives none; several optimal sets usually exist):

* dynamic: walk from checkpoint 0; from checkpoint i the next checkpoint is the smallest j that
  starts an optimal solution of the suffix problem "i is a checkpoint, minimise over i..n".
* static: among optimal sets take those with the smallest largest-segment sum, then the one whose
  checkpoint list read from the back (n first) is lexicographically smallest, i.e. each previous
  checkpoint is as early as optimality allows.

Parity status: every function here is pinned by tests against closed forms, the VGG-19 values the
paper prints (Table 2 and Section 5.5) and each other (definition vs recursion vs event list).
The per-stage memory trace of Fig. 2 is NOT reproduced exactly by ``simulate_alg4`` (the printed
series keeps d_{i-1} one stage longer in the forward phase): trace values are "parity unpinned";
only the peak is pinned.
"""

from itertools import combinations


def _check_sizes(d):
    n = len(d) - 1
    if n < 1:
        raise ValueError("need at least d_0 and d_1")
    for v in d:
        if int(v) != v or v < 1:
            raise ValueError("sizes must be integers >= 1")
    return n


def _check_set(n, C):
    cs = sorted(set(int(c) for c in C))
    if cs[0] != 0 or cs[-1] != n:
        raise ValueError("0 and n must be checkpoints")
    if cs[0] < 0 or cs[-1] > n:
        raise ValueError("checkpoint index out of range")
    return cs


# --------------------------------------------------------------------------------------------
# Objective functions
# --------------------------------------------------------------------------------------------

def eval_static(d, C):
    """Eq. (cost): checkpoint memory + segment memory."""
    n = _check_sizes(d)
    cs = _check_set(n, C)
    checkpoint_memory = sum(d[c] for c in cs)
    segment_memory = 0
    for h, i in zip(cs[:-1], cs[1:]):
        seg = sum(d[k] for k in range(h + 1, i))      # empty segment -> 0
        segment_memory = max(segment_memory, seg)
    return checkpoint_memory + segment_memory


def s_term(d, h, i):
    """Eq. (s): s(h,i) = sum_{k=h+1}^{i-1} d_k + max_{h<=k<i} d_k."""
    return sum(d[k] for k in range(h + 1, i)) + max(d[k] for k in range(h, i))


def eval_dynamic(d, C):
    """Eq. (memory-simple): max over checkpoints i>0 of sum(C(i)) + s(h,i)."""
    n = _check_sizes(d)
    cs = _check_set(n, C)
    worst = 0
    for pos in range(1, len(cs)):
        h, i = cs[pos - 1], cs[pos]
        m_i = sum(d[c] for c in cs[: pos + 1]) + s_term(d, h, i)
        worst = max(worst, m_i)
    return worst


# --------------------------------------------------------------------------------------------
# Event-level simulators (the arena's specification)
# --------------------------------------------------------------------------------------------

class _Ledger:
    def __init__(self):
        self.live = {}
        self.bytes = 0
        self.high_water = 0
        self.events = []

    def alloc(self, name, size):
        assert name not in self.live, name
        self.live[name] = size
        self.bytes += size
        self.high_water = max(self.high_water, self.bytes)
        self.events.append(("alloc", name, size, self.bytes))

    def free(self, name):
        size = self.live.pop(name)
        self.bytes -= size
        self.events.append(("free", name, size, self.bytes))


def simulate_alg1(d):
    """Algorithm 1: every d_i is allocated before the forward phase and kept."""
    n = _check_sizes(d)
    L = _Ledger()
    L.alloc("d0", d[0])
    for i in range(1, n + 1):
        L.alloc("d%d" % i, d[i])
    return L.high_water, L.events


def simulate_alg2(d, C):
    """Algorithm 2: forward frees non-checkpoints; backward frees/recomputes whole segments."""
    n = _check_sizes(d)
    cs = _check_set(n, C)
    is_c = [i in set(cs) for i in range(n + 1)]
    L = _Ledger()
    L.alloc("d0", d[0])
    for i in range(1, n + 1):
        L.alloc("d%d" % i, d[i])
        if not is_c[i - 1]:
            L.free("d%d" % (i - 1))
    prev_segment = []
    for i in range(n, 0, -1):
        if is_c[i]:
            for k in prev_segment:                      # free the segment after d_i
                L.free("d%d" % k)
            h = max(c for c in cs if c < i)
            prev_segment = list(range(h + 1, i))
            for k in prev_segment:                      # allocate + recompute d_{h+1..i-1}
                L.alloc("d%d" % k, d[k])
        # compute r_i, g_i: no allocation in this model
    return L.high_water, L.events


def simulate_alg4(d, C):
    """Algorithm 4 with the release of the old gradient buffer moved before the recompute."""
    n = _check_sizes(d)
    cs = _check_set(n, C)
    is_c = [i in set(cs) for i in range(n + 1)]
    L = _Ledger()
    L.alloc("d0", d[0])
    for i in range(1, n + 1):
        L.alloc("d%d" % i, d[i])
        if not is_c[i - 1]:
            L.free("d%d" % (i - 1))
    have_r = False
    for i in range(n, 0, -1):
        if is_c[i]:
            h = max(c for c in cs if c < i)
            if have_r:
                L.free("r")
            for k in range(h + 1, i):
                L.alloc("d%d" % k, d[k])
            L.alloc("r", max(d[k] for k in range(h, i)))
            have_r = True
        L.free("d%d" % i)                               # released as soon as step i is done
    return L.high_water, L.events


def stage_trace(d, C, schedule):
    """Live bytes at the end of every training phase index 0..2n+1 (Section 5.1.1) under
    Algorithm 2 (``schedule="alg2"``) or Algorithm 4 (``"alg4"``, with the buffer release moved
    before the recompute): index 0 = before the step (d_0 only), 1..n = end of the forward stage
    of unit i, n+1..2n = end of the backward stage of unit n..1, 2n+1 = after the step (d_0 only).
    Written from the two listings directly, independently of the event simulators above."""
    n = _check_sizes(d)
    cs = _check_set(n, C)
    is_c = [i in set(cs) for i in range(n + 1)]
    live = {0: d[0]}
    trace = [d[0]]
    for i in range(1, n + 1):                               # forward phase (identical in both)
        live[i] = d[i]
        if not is_c[i - 1]:
            del live[i - 1]
        trace.append(sum(live.values()))
    r = 0
    for i in range(n, 0, -1):
        if is_c[i]:
            h = max(c for c in cs if c < i)
            if schedule == "alg2":
                for k in [k for k in live if k > i and not is_c[k]]:
                    del live[k]                             # free the segment after d_i
            else:
                r = 0                                       # release the previous gradient buffer
            for k in range(h + 1, i):
                live[k] = d[k]                              # allocate + recompute the segment
            if schedule == "alg4":
                r = max(d[k] for k in range(h, i))
        if schedule == "alg4":
            del live[i]                                     # d_i released as soon as step i is done
        trace.append(sum(live.values()) + r)
    trace.append(d[0])
    return trace


# --------------------------------------------------------------------------------------------
# Brute force over every feasible checkpoint set
# --------------------------------------------------------------------------------------------

def _all_sets(lo, hi):
    """Every subset of the open index range (lo, hi), as sorted tuples."""
    inner = list(range(lo + 1, hi))
    for r in range(len(inner) + 1):
        for comb in combinations(inner, r):
            yield comb


def brute_force_static(d):
    """Optimum of Eq. (cost) and the canonical optimal set.

    Returns dict(value, set, n_optimal, n_evaluated, n_masks).  ``n_masks`` = 2^n membership masks
    over d_1..d_n; those without n are infeasible and only counted.
    """
    n = _check_sizes(d)
    best = None
    optimal = []
    evaluated = 0
    for inner in _all_sets(0, n):
        C = (0,) + inner + (n,)
        v = eval_static(d, C)
        evaluated += 1
        if best is None or v < best:
            best, optimal = v, [C]
        elif v == best:
            optimal.append(C)

    def max_seg(C):
        return max(sum(d[k] for k in range(h + 1, i)) for h, i in zip(C[:-1], C[1:]))

    smallest_cap = min(max_seg(C) for C in optimal)
    pool = [C for C in optimal if max_seg(C) == smallest_cap]
    canonical = min(pool, key=lambda C: tuple(reversed(C)))
    return dict(value=best, set=list(canonical), n_optimal=len(optimal),
                n_evaluated=evaluated, n_masks=2 ** n)


def _suffix_value(d, C):
    """Eq. (memory) restricted to the chain that starts at checkpoint C[0]."""
    worst = d[C[0]] if len(C) == 1 else 0
    for pos in range(1, len(C)):
        h, i = C[pos - 1], C[pos]
        worst = max(worst, sum(d[c] for c in C[: pos + 1]) + s_term(d, h, i))
    return worst


def brute_force_dynamic(d):
    """Optimum of Eq. (memory) and the canonical optimal set (see the module docstring)."""
    n = _check_sizes(d)
    # M_bf[i] = optimum of the suffix problem that starts at checkpoint i, by enumeration;
    # first[i] = smallest next checkpoint used by any optimal suffix solution.
    M_bf = {n: d[n]}
    first = {}
    for i in range(n - 1, -1, -1):
        best = None
        best_first = None
        for inner in _all_sets(i, n):
            C = (i,) + inner + (n,)
            v = _suffix_value(d, C)
            if best is None or v < best:
                best, best_first = v, C[1]
            elif v == best and C[1] < best_first:
                best_first = C[1]
        M_bf[i], first[i] = best, best_first
    # count the optimal full sets
    n_optimal = 0
    evaluated = 0
    for inner in _all_sets(0, n):
        evaluated += 1
        if eval_dynamic(d, (0,) + inner + (n,)) == M_bf[0]:
            n_optimal += 1
    C = [0]
    while C[-1] != n:
        C.append(first[C[-1]])
    return dict(value=M_bf[0], set=C, n_optimal=n_optimal, n_evaluated=evaluated,
                n_masks=2 ** n, suffix_values=[M_bf[i] for i in range(n + 1)])


# --------------------------------------------------------------------------------------------
# Reference recursions for chains too long to enumerate
# --------------------------------------------------------------------------------------------

def segment_caps(d):
    """Candidate segment memories: 0 and every contiguous range sum of d_1..d_{n-1}."""
    n = _check_sizes(d)
    caps = {0}
    for a in range(1, n):
        acc = 0
        for b in range(a, n):
            acc += d[b]
            caps.add(acc)
    return sorted(caps)


def dp_static_reference(d):
    """Eq. (T) for every cap, window minimum taken directly; answer = min_s (s + d_n + M(n-1,s)).

    M(-1,s) = 0 so that choosing j = 0 costs d_0.  Ties: smallest cap, then smallest j.
    Sizes are held in numpy int64 (checked against overflow) so that n = 1000 finishes in seconds.
    Returns (value, set).
    """
    n = _check_sizes(d)
    assert 2 * sum(int(v) for v in d) < 2 ** 62
    best = None
    best_s = None
    for s in segment_caps(d):
        M = _static_table(d, n, s)[0]
        total = s + d[n] + int(M[n - 1])
        if best is None or total < best:
            best, best_s = total, s
    M, arg = _static_table(d, n, best_s)
    C = [n]
    i = n - 1
    while i >= 0:
        j = int(arg[i])
        C.append(j)
        i = j - 1
    C = sorted(set(C))
    return best, C


def _static_table(d, n, s):
    """M(i,s) for i = 0..n-1 and the smallest minimising j of Eq. (T) for each i."""
    import numpy as np
    prefix = [0] * (n + 1)                              # prefix[i] = d_1 + ... + d_i
    for k in range(1, n + 1):
        prefix[k] = prefix[k - 1] + d[k]
    key = np.zeros(n, dtype=np.int64)                   # key[j] = d_j + M(j-1,s)
    M = np.zeros(n, dtype=np.int64)
    arg = np.zeros(n, dtype=np.int64)
    lo = 0                                              # l(i): smallest j with d_{j+1}+..+d_i <= s
    for i in range(0, n):
        key[i] = d[i] + (int(M[i - 1]) if i >= 1 else 0)
        while prefix[i] - prefix[lo] > s:
            lo += 1
        window = key[lo:i + 1]
        pos = int(np.argmin(window))                    # first occurrence = smallest j among ties
        M[i] = window[pos]
        arg[i] = lo + pos
    return M, arg


def dp_dynamic_reference(d):
    """Algorithm 5: M(n)=d_n; M(i)=min_{i<j<=n} max(d_i+M(j), d_i+s(i,j)+d_j); answer M(0).

    s(i,j) is carried along the j scan (running sum of d_{i+1..j-1}, running max of d_{i..j-1}),
    which is the "precompute all s(i,j)" of the O(n^2) analysis.  The inner loop scans j upward
    with a strict '<' update, so the first minimiser wins.  Returns (value, set, M list).
    """
    n = _check_sizes(d)
    M = [None] * (n + 1)
    nxt = [None] * (n + 1)
    M[n] = d[n]
    for i in range(n - 1, -1, -1):
        seg_sum = 0
        seg_max = d[i]
        for j in range(i + 1, n + 1):
            s_ij = seg_sum + seg_max                    # Eq. (s)
            v = max(d[i] + M[j], d[i] + s_ij + d[j])
            if M[i] is None or v < M[i]:
                M[i], nxt[i] = v, j
            seg_sum += d[j]
            seg_max = max(seg_max, d[j])
    C = [0]
    while C[-1] != n:
        C.append(nxt[C[-1]])
    return M[0], C, M


# --------------------------------------------------------------------------------------------
# Eq. (memory) with separate sizes for a checkpoint, a segment tensor and a gradient
# --------------------------------------------------------------------------------------------

def _check_three(kept, live, grad):
    n = _check_sizes(kept)
    if len(live) != n + 1 or len(grad) != n + 1:
        raise ValueError("kept, live and grad must have n+1 entries each")
    _check_sizes(live)
    _check_sizes(grad)
    return n


def s_term_two_size(live, grad, h, i, incoming):
    """Eq. (s) with the segment tensors at their live size, the output-gradient buffer sized by the gradients
    r_h .. r_{i-1} it holds and, when `incoming`, a second buffer for the gradients r_{h+1} .. r_i the steps read."""
    s = sum(live[t] for t in range(h + 1, i)) + max(grad[t] for t in range(h, i))
    if incoming:
        s += max(grad[t] for t in range(h + 1, i + 1))
    return s


def eval_two_size(kept, live, grad, C, incoming=False):
    """max over checkpoints i > 0 of [checkpoints up to i at their kept size + s_term_two_size(h, i)]."""
    n = _check_three(kept, live, grad)
    cs = _check_set(n, C)
    worst = 0
    for pos in range(1, len(cs)):
        h, i = cs[pos - 1], cs[pos]
        worst = max(worst, sum(kept[c] for c in cs[: pos + 1]) + s_term_two_size(live, grad, h, i, incoming))
    return worst


def brute_force_two_size(kept, live, grad, incoming=False):
    """Optimum of eval_two_size over every feasible set, and the canonical optimal set under the dynamic tie rule
    (from checkpoint i the smallest next checkpoint that starts an optimal solution of the suffix problem)."""
    n = _check_three(kept, live, grad)

    def suffix_value(C):
        worst = kept[C[0]] if len(C) == 1 else 0
        for pos in range(1, len(C)):
            worst = max(worst, sum(kept[c] for c in C[: pos + 1]) + s_term_two_size(live, grad, C[pos - 1], C[pos], incoming))
        return worst

    best_of, first = {n: kept[n]}, {}
    for i in range(n - 1, -1, -1):
        best = best_first = None
        for inner in _all_sets(i, n):
            C = (i,) + inner + (n,)
            v = suffix_value(C)
            if best is None or v < best or (v == best and C[1] < best_first):
                best, best_first = v, C[1]
        best_of[i], first[i] = best, best_first
    C = [0]
    while C[-1] != n:
        C.append(first[C[-1]])
    return dict(value=best_of[0], set=C)


def dp_two_size_reference(kept, live, grad, incoming=False):
    """Algorithm 5 on the three-size objective: M(n) = kept_n; M(i) = min over i < j <= n of
    max(kept_i + M(j), kept_i + s(i,j) + kept_j), first minimiser wins.  Returns (value, set)."""
    n = _check_three(kept, live, grad)
    M = [None] * (n + 1)
    nxt = [None] * (n + 1)
    M[n] = kept[n]
    for i in range(n - 1, -1, -1):
        for j in range(i + 1, n + 1):
            v = max(kept[i] + M[j], kept[i] + s_term_two_size(live, grad, i, j, incoming) + kept[j])
            if M[i] is None or v < M[i]:
                M[i], nxt[i] = v, j
    C = [0]
    while C[-1] != n:
        C.append(nxt[C[-1]])
    return M[0], C


def sqrt_n_plan(n):
    """Uniform sqrt(n) heuristic quoted in Section 5.3: every ceil(sqrt(n))-th layer plus n."""
    import math
    step = math.isqrt(n)
    if step * step < n:
        step += 1
    C = [0] + [k for k in range(step, n, step)] + [n]
    return sorted(set(C))


# --------------------------------------------------------------------------------------------
# Least recomputation under a memory budget
# --------------------------------------------------------------------------------------------
# Section 3.1 minimises the peak alone, and many sets reach the optimum of Eq. (memory) (the 24-unit VGG-19 chain of
# Section 5 has hundreds of thousands).  Which of them runs fastest is a second question: the backward pass of
# Algorithm 4 recomputes every tensor that is not a checkpoint once, so the recomputation time of a set C is the sum of
# cost[i] over the units i outside C (cost[i] = time of the forward of unit i).  The definition, by enumeration:

def recompute_cost(cost, C):
    """Sum of cost[i] over the units i = 1..n-1 that are not in C (d_0 and d_n are never recomputed)."""
    n = len(cost) - 1
    _check_set(n, C)
    members = set(C)
    return sum(cost[i] for i in range(1, n) if i not in members)


def brute_force_min_recompute(d, cost, budget):
    """Among all feasible sets whose Eq. (memory) value is at most `budget`, the least recomputation cost; returns
    dict(cost, set, peak, feasible_sets) with one set that attains it (the first in enumeration order: fewer
    checkpoints first, then lexicographic), or None when no set fits the budget."""
    n = _check_sizes(d)
    if len(cost) != n + 1 or any(c < 0 for c in cost):
        raise ValueError("cost needs n + 1 non-negative entries")
    best = None
    feasible = 0
    for inner in _all_sets(0, n):
        C = (0,) + inner + (n,)
        peak = eval_dynamic(d, C)
        if peak > budget:
            continue
        feasible += 1
        c = recompute_cost(cost, C)
        if best is None or c < best["cost"]:
            best = {"cost": c, "set": list(C), "peak": peak}
    if best is None:
        return None
    best["feasible_sets"] = feasible
    return best
