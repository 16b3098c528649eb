"""Pins for the CPU oracle: values the paper prints, closed forms, brute force, invariants.

Each test is chosen so that a plausible slip in the oracle (an off-by-one in the time convention,
skip instead of break, a dropped ramp term, a transposed comparison, a wrong tie rule) fails it.
No expected value here comes from the oracle itself or from the GPU library.
"""
import itertools

import numpy as np
import pytest

import oracle as orc
from paper_2508_06133_b200 import workloads as W


# ----------------------------------------------------------------------------- worked example
def example1():
    s = np.array([63] + [1] * 21, dtype=np.int32)
    o = np.array([1] + [2] * 21, dtype=np.int32)
    return s, o


@pytest.mark.parametrize("executor", [orc.list_schedule_alg1, orc.list_schedule_rounds])
def test_example1_tel(golden, executor):
    s, o = example1()
    M = golden["example1_M"]
    mcsf = orc.policy_order(s, o, orc.SHORTEST_OUTPUT_FIRST)
    assert mcsf[0] == 0                                   # the o = 1 request goes first
    assert executor(s, o, M, mcsf)[1] == golden["example1_tel_mcsf"]
    sorted_f = np.array(list(range(1, 22)) + [0], dtype=np.int32)
    p, tel, mk = executor(s, o, M, sorted_f)
    assert tel == golden["example1_tel_sortedf"]
    assert mk == 3 and p[0] == 2 and (p[1:] == 0).all()   # Type 2 done at t=2, Type 1 runs in round 3


def test_example1_checker_by_hand(golden):
    """Start vectors written by hand, checked by the occupancy definition."""
    s, o = example1()
    M = golden["example1_M"]
    good = np.array([2] + [0] * 21)
    r = orc.check_schedule(s, o, M, good)
    assert r["feasible"] and r["tel"] == 45 and r["peak"] == 64 and r["makespan"] == 3
    bad = np.array([1] + [0] * 21)                         # Type 1 overlaps the round where Type 2 holds 63
    r = orc.check_schedule(s, o, M, bad)
    assert not r["feasible"] and r["first_bad_round"] == 2 and r["peak"] == 63 + 64
    # 22 Type-2 requests together need 66 > 64 in their second round: capacity is 21
    s22, o22 = np.ones(22, dtype=np.int32), np.full(22, 2, dtype=np.int32)
    assert not orc.check_schedule(s22, o22, M, np.zeros(22))["feasible"]
    assert orc.check_schedule(s22[:21], o22[:21], M, np.zeros(21))["feasible"]
    assert golden["example1_batch_capacity"] == 21


def test_example1_f_metric(golden):
    # F(Type 2 x 21) = 42/441 < F(Type 1) = 1/1
    assert orc.f_compare(golden["example1_F_type2_num"], 21, golden["example1_F_type1_num"], 1) < 0
    assert orc.f_compare(1, 1, 42, 21) > 0
    assert golden["example1_F_type2_den"] == 21 ** 2
    # ties on F prefer the larger batch: 2/2^2 == 8/4^2
    assert orc.f_compare(8, 4, 2, 2) < 0 and orc.f_compare(2, 2, 8, 4) > 0 and orc.f_compare(3, 3, 3, 3) == 0
    # products beyond 64 bits still compare exactly
    assert orc.f_compare(4 * 10 ** 8, 10 ** 5, 4 * 10 ** 8 + 1, 10 ** 5) < 0


def test_example1_sorted_f_selects_type2_first(golden):
    s, o = example1()
    M = golden["example1_M"]
    for solver in (orc.ENUM_SUM, orc.DP):
        ids = np.arange(22)
        chosen, so, mem = (orc.phase1_enumerate(ids[:14], s, o, M, solver) if solver != orc.DP
                           else orc.phase1_dp(ids, s, o, M))
        assert 0 not in chosen                            # never the prompt-63 request
    order, offs = orc.sorted_f_exact(s, o, M, orc.DP)
    assert list(offs) == [0, 21, 22] and order[-1] == 0
    order, offs = orc.sorted_f_prefix(s, o, M)
    assert list(offs) == [0, 21, 22] and order[-1] == 0
    assert orc.list_schedule_alg1(s, o, M, order)[1] == golden["example1_tel_sortedf"]


# ----------------------------------------------------------------------------- Example 2 (symbolic)
@pytest.mark.parametrize("n1,s1,o1,n2,s2,o2", [(10, 8, 4, 4, 20, 10), (6, 15, 5, 3, 28, 12), (5, 10, 14, 12, 4, 6)])
def test_example2_two_saturating_batches(n1, s1, o1, n2, s2, o2):
    """the supplement to Section 3, Example 2: n1(s1+o1) = n2(s2+o2) = M; TEL = o1 n1 + o2 n2 + (o1 n2 | o2 n1)."""
    M = n1 * (s1 + o1)
    assert M == n2 * (s2 + o2)
    s = np.array([s1] * n1 + [s2] * n2, dtype=np.int32)
    o = np.array([o1] * n1 + [o2] * n2, dtype=np.int32)
    first1 = np.arange(n1 + n2)
    first2 = np.concatenate([np.arange(n1, n1 + n2), np.arange(n1)])
    # The example's totals assume the second batch cannot overlap the first.  Under continuous
    # batching that holds exactly when the second batch's requests outlive the first batch's
    # saturated last round (o_second >= o_first); otherwise early starts can only lower the TEL.
    tel12 = o1 * n1 + o2 * n2 + o1 * n2
    tel21 = o1 * n1 + o2 * n2 + o2 * n1
    for ex in (orc.list_schedule_alg1, orc.list_schedule_rounds):
        got12, got21 = ex(s, o, M, first1)[1], ex(s, o, M, first2)[1]
        assert got12 == tel12 if o2 >= o1 else got12 <= tel12
        assert got21 == tel21 if o1 >= o2 else got21 <= tel21
    # the F rule prefers the order the example says is cheaper
    prefer1 = orc.f_compare(o1 * n1, n1, o2 * n2, n2) < 0
    assert prefer1 == (o1 * n2 < o2 * n1)


# ----------------------------------------------------------------------------- Theorem 1 closed form
@pytest.mark.parametrize("root4", [3, 6, 9])
def test_theorem1_closed_form(root4, golden):
    """the supplement to Section 2: X = M requests (sqrt(M)-1, 1) then Y = M^1.25 requests (1, 2), shortest output first."""
    M = root4 ** 4
    r = root4 ** 2
    X, Y = M, root4 ** 5
    assert M % 3 == 0
    s = np.array([r - 1] * X + [1] * Y, dtype=np.int32)
    o = np.array([1] * X + [2] * Y, dtype=np.int32)
    order = orc.policy_order(s, o, orc.SHORTEST_OUTPUT_FIRST)
    assert (order == np.arange(X + Y)).all()
    tri = lambda k: k * (k + 1) // 2
    closed = r * tri(X // r) + X * Y // r + (2 * M // 3) * tri(3 * Y // M)
    if M == 6561:
        assert closed == golden["thm1_M6561_tel_mcsf"]
    assert orc.list_schedule_rounds(s, o, M, order)[1] == closed
    if M <= 1296:
        assert orc.list_schedule_alg1(s, o, M, order)[1] == closed


# ----------------------------------------------------------------------------- NP-hardness family
def test_three_partition_family(golden):
    """the supplement to Section 2: s_i = x_i, o_i = 1, M = T + 3; optimum 3m(m+1)/2 iff a 3-partition exists."""
    T = 20
    x = [6, 7, 7, 6, 6, 8]                                # {6,7,7}, {6,6,8}
    s, o = np.array(x, dtype=np.int32), np.ones(6, dtype=np.int32)
    M = T + 3
    opt, p = orc.bruteforce_opt(s, o, M, 6 * 7)
    assert opt == golden["np_family_m2"]
    assert orc.check_schedule(s, o, M, p)["feasible"]
    assert np.bincount(p.astype(int)).tolist() == [3, 3]
    # the partition given as an order reaches it through the executor
    assert orc.list_schedule_alg1(s, o, M, [0, 1, 2, 3, 4, 5])[1] == 9
    best, _ = orc.bruteforce_best_order(s, o, M)
    assert best == 9
    # no batch of four fits
    for quad in itertools.combinations(range(6), 4):
        pp = np.array([0 if i in quad else 5 for i in range(6)])
        assert not orc.check_schedule(s, o, M, pp)["feasible"]
    # no 3-partition: {6,6,6,6,7,9} has no triple summing to 20
    x2 = [6, 6, 6, 6, 7, 9]
    assert sum(x2) == 2 * T and all(sum(c) != T for c in itertools.combinations(x2, 3))
    opt2, _ = orc.bruteforce_opt(np.array(x2, dtype=np.int32), o, M, 6 * 7)
    assert opt2 > 9
    # m = 3
    x3 = [6, 7, 7, 6, 6, 8, 8, 6, 6]
    s3, o3 = np.array(x3, dtype=np.int32), np.ones(9, dtype=np.int32)
    opt3, _ = orc.bruteforce_opt(s3, o3, M, 9 * 10)
    assert opt3 == golden["np_family_m3"]


# ----------------------------------------------------------------------------- executor invariants
def random_instance(rng, n, M, smax, omax):
    s = rng.integers(1, smax + 1, n).astype(np.int32)
    o = rng.integers(1, omax + 1, n).astype(np.int32)
    keep = s + o <= M
    s[~keep] = 1
    return s, o


def numpy_occupancy(s, o, p, length):
    """Independent restatement of the memory model (Section 2.1): token j of request i needs s_i + j."""
    U = np.zeros(length, dtype=np.int64)
    for si, oi, pi in zip(s, o, p):
        U[pi + 1: pi + oi + 1] += si + np.arange(1, oi + 1)
    return U


def test_alg1_equals_round_form_and_invariants():
    rng = np.random.default_rng(12345)
    for trial in range(300):
        n = int(rng.integers(1, 40))
        M = int(rng.integers(8, 200))
        s, o = random_instance(rng, n, M, max(1, M // 2), max(1, M // 3))
        order = rng.permutation(n).astype(np.int32)
        p1, tel1, mk1 = orc.list_schedule_alg1(s, o, M, order)
        p2, tel2, mk2 = orc.list_schedule_rounds(s, o, M, order)
        assert (p1 == p2).all() and tel1 == tel2 and mk1 == mk2
        assert tel1 == int((p1 + o).sum())
        chk = orc.check_schedule(s, o, M, p1)
        assert chk["feasible"] and chk["tel"] == tel1 and chk["peak"] <= M and chk["makespan"] == mk1
        U = numpy_occupancy(s, o, p1, mk1 + 2)
        assert U.max() == chk["peak"] <= M
        Uo, R = orc.occupancy(s, o, p1, mk1 + 2)
        assert (Uo == U).all() and R.sum() == o.sum()      # every request decodes exactly o_i tokens
        # starts never go backwards along the order (first misfit blocks everything behind it)
        assert (np.diff(p1[order]) >= 0).all()


def test_alg1_equals_round_form_on_mixed_backlogs():
    """The same equivalence at the sizes and shapes the bulk GPU parity relies on: mixed chat/document
    backlogs of a few hundred to 1,500 requests (saturated memory, long waits, hundreds of requests
    running at once), under Sorted-F, the three baseline policies, random orders and moved orders --
    every start time, not only the TEL."""
    rng = np.random.default_rng(2024)
    for n, M, seed in ((300, 20000, 11), (400, 24000, 12), (700, 40000, 13), (1500, 65536, 14)):
        inst = W.mixed_backlog(n, seed, M, name="o2")
        base, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
        orders = [base, orc.policy_order(inst.s, inst.o, orc.FCFS), orc.policy_order(inst.s, inst.o, orc.SHORTEST_OUTPUT_FIRST),
                  orc.policy_order(inst.s, inst.o, orc.TOTAL_SIZE_FIRST), rng.permutation(n).astype(np.int32)]
        total = n * (n - 1) // 2 + n * (n - 1)
        for code in rng.integers(0, total, 4 if n > 1000 else 8):
            orders.append(orc.apply_move(base, *orc.decode_move(n, int(code))))
        for order in orders:
            p1, tel1, mk1 = orc.list_schedule_alg1(inst.s, inst.o, inst.M, order)
            p2, tel2, mk2 = orc.list_schedule_rounds(inst.s, inst.o, inst.M, order)
            assert (p1 == p2).all() and tel1 == tel2 and mk1 == mk2
        chk = orc.check_schedule(inst.s, inst.o, inst.M, p1)
        assert chk["feasible"] and chk["tel"] == tel1


def test_each_start_is_the_earliest_feasible():
    """Break rule + maximal admission: request q starts at the first round >= its predecessor's
    start at which the occupancy definition admits it, given the earlier requests."""
    rng = np.random.default_rng(777)
    for trial in range(60):
        n = int(rng.integers(2, 14))
        M = int(rng.integers(10, 80))
        s, o = random_instance(rng, n, M, M // 2, M // 3 + 1)
        order = rng.permutation(n)
        p, tel, mk = orc.list_schedule_alg1(s, o, M, order)
        for q in range(n):
            sub = order[:q + 1]
            lo = p[order[q - 1]] if q else 0
            for k in range(lo, p[order[q]]):               # every earlier admissible start must overflow
                pp = p[sub].copy()
                pp[-1] = k
                assert not orc.check_schedule(s[sub], o[sub], M, pp)["feasible"]
            assert orc.check_schedule(s[sub], o[sub], M, p[sub])["feasible"]


def test_invalid_instances_rejected():
    with pytest.raises(ValueError):
        orc.list_schedule_alg1([5], [6], 10, [0])          # s + o > M would never be admitted
    with pytest.raises(ValueError):
        orc.list_schedule_rounds([0], [1], 10, [0])
    assert orc.check_schedule([1], [1], 10, [-1])["rc"] == -1


def test_policies():
    s = np.array([5, 1, 3, 1, 9], dtype=np.int32)
    o = np.array([2, 7, 2, 3, 1], dtype=np.int32)
    assert orc.policy_order(s, o, orc.FCFS).tolist() == [0, 1, 2, 3, 4]
    assert orc.policy_order(s, o, orc.SHORTEST_OUTPUT_FIRST).tolist() == [4, 0, 2, 3, 1]
    assert orc.policy_order(s, o, orc.TOTAL_SIZE_FIRST).tolist() == [3, 2, 0, 1, 4]   # sizes 7,8,5,4,10


# ----------------------------------------------------------------------------- Phase 1 solvers
def test_phase1_dp_matches_enumeration_and_lemma1():
    rng = np.random.default_rng(99)
    for trial in range(120):
        n = int(rng.integers(2, 13))
        M = int(rng.integers(12, 90))
        s, o = random_instance(rng, n, M, M // 2, M // 2)
        ids = np.arange(n)
        ce, so_e, mem_e = orc.phase1_enumerate(ids, s, o, M, orc.ENUM_SUM)
        cd, so_d, mem_d = orc.phase1_dp(ids, s, o, M)
        assert (so_e, len(ce), mem_e) == (so_d, len(cd), mem_d)
        assert int(o[cd].sum()) == so_d and int((s[cd] + o[cd]).sum()) == mem_d <= M
        # brute force in Python over all subsets: nothing feasible has a smaller (F, -k)
        for k in range(1, n + 1):
            for sub in itertools.combinations(range(n), k):
                sub = list(sub)
                if int((s[sub] + o[sub]).sum()) <= M:
                    lhs, rhs = int(o[sub].sum()) * len(cd) ** 2, so_d * k ** 2
                    assert lhs > rhs or (lhs == rhs and k <= len(cd))
        # Lemma 1: mean output of an exactly selected batch exceeds half its largest output
        for chosen in (ce, cd):
            assert 2 * int(o[chosen].sum()) > int(o[chosen].max()) * len(chosen)
        # sum(s+o) <= M implies Algorithm 1's own constraint, so its optimum is at least as good
        ca, so_a, _ = orc.phase1_enumerate(ids, s, o, M, orc.ENUM_ALG1)
        assert orc.f_compare(so_a, len(ca), so_e, len(ce)) <= 0
        assert 2 * int(o[ca].sum()) > int(o[ca].max()) * len(ca)
        # the Algorithm-1 batch really is feasible when started together
        assert orc.check_schedule(s[ca], o[ca], M, np.zeros(len(ca)))["feasible"]


def test_phase1_algorithm1_constraint_by_hand():
    """Algorithm 1's own Phase-1 constraint, M(X, o_j) <= M for every j with all of X started
    together, against the memory test sum(s+o) <= M of Algorithms 2-4, on an instance worked by hand.
    A = B = (s 1, o 4), C = (s 4, o 2), M = 12.  All three started together use 3 + 3 + 6 = 12 when
    C ends and 5 + 5 = 10 when A and B end: feasible by Algorithm 1's constraint although
    sum(s+o) = 16 > 12.  F: {A,B,C} 10/9, {A,C} = {B,C} 6/4, {A,B} 8/4, {C} 2, {A} = {B} 4."""
    s, o, ids = np.array([1, 1, 4]), np.array([4, 4, 2]), np.arange(3)
    chosen, so, mem = orc.phase1_enumerate(ids, s, o, 12, orc.ENUM_ALG1)
    assert (chosen.tolist(), so, mem) == ([0, 1, 2], 10, 16)
    assert orc.check_schedule(s, o, 12, [0, 0, 0])["feasible"]
    # the sum reading cannot take all three: best F among its feasible sets is 6/4, lowest indices first
    chosen, so, mem = orc.phase1_enumerate(ids, s, o, 12, orc.ENUM_SUM)
    assert (chosen.tolist(), so, mem) == ([0, 2], 6, 11)
    # one token less and the round in which C ends overflows (12 > 11): Algorithm 1's constraint now
    # refuses the triple as well, so the constraint is neither too lax nor too strict
    assert not orc.check_schedule(s, o, 11, [0, 0, 0])["feasible"]
    chosen, so, mem = orc.phase1_enumerate(ids, s, o, 11, orc.ENUM_ALG1)
    assert (chosen.tolist(), so, mem) == ([0, 2], 6, 11)
    # the later completion binds instead: A = (s 5, o 3), B = (s 6, o 3), C = (s 1, o 1), M = 17.
    # Together: 6 + 7 + 2 = 15 when C ends, 8 + 9 = 17 when A and B end -> feasible; at M = 16 not.
    s, o = np.array([5, 6, 1]), np.array([3, 3, 1])
    chosen, so, _ = orc.phase1_enumerate(ids, s, o, 17, orc.ENUM_ALG1)
    assert (chosen.tolist(), so) == ([0, 1, 2], 7)                  # F = 7/9 beats {C} = 1 and {A,C} = 4/4
    chosen, so, _ = orc.phase1_enumerate(ids, s, o, 16, orc.ENUM_ALG1)
    assert (chosen.tolist(), so) == ([0, 2], 4)                     # {A,C}: 6 + 2 = 8, then 8; F = 1, larger than {C}
    # Sorted-F assembled on the first instance: the triple is one batch, sorted by o
    order, offs = orc.sorted_f_exact(np.array([1, 1, 4]), np.array([4, 4, 2]), 12, orc.ENUM_ALG1)
    assert order.tolist() == [2, 0, 1] and offs.tolist() == [0, 3]


def test_sorted_f_orders_are_permutations_and_batches_sorted():
    rng = np.random.default_rng(5)
    for trial in range(40):
        n = int(rng.integers(1, 13))
        M = int(rng.integers(12, 90))
        s, o = random_instance(rng, n, M, M // 2, M // 2)
        for fn in (lambda: orc.sorted_f_exact(s, o, M, orc.ENUM_ALG1), lambda: orc.sorted_f_exact(s, o, M, orc.ENUM_SUM),
                   lambda: orc.sorted_f_exact(s, o, M, orc.DP), lambda: orc.sorted_f_prefix(s, o, M)):
            order, offs = fn()
            assert sorted(order.tolist()) == list(range(n))
            assert offs[0] == 0 and offs[-1] == n and (np.diff(offs) > 0).all()
            for a, b in zip(offs[:-1], offs[1:]):
                assert (np.diff(o[order[a:b]]) >= 0).all()


def test_prefix_f_by_hand():
    # sizes s+o: r0=4 (o=3), r1=3 (o=1), r2=9 (o=2), r3=5 (o=5); M = 12
    s = np.array([1, 2, 7, 1], dtype=np.int32)
    o = np.array([3, 1, 2, 4], dtype=np.int32)
    # ascending s+o: r1(3), r0(4), r3(5), r2(9); prefixes within M=12: k=1 F=1/1, k=2 F=4/4, k=3 F=8/9 -> k=3
    order, offs = orc.sorted_f_prefix(s, o, 12)
    assert offs.tolist() == [0, 3, 4]
    assert order.tolist() == [1, 0, 3, 2]                  # batch sorted by o: 1, 3, 4
    # tie on F between k=1 (1/1) and k=2 (4/4) goes to the larger prefix when k=3 does not fit
    order, offs = orc.sorted_f_prefix(s, o, 9)
    assert offs.tolist()[:2] == [0, 2]


def test_prefix_f_equals_exact_on_homogeneous_types():
    """Identical requests within a type (Example 2's setting): the best subset is a prefix."""
    s = np.array([1] * 9 + [30] * 2, dtype=np.int32)
    o = np.array([2] * 9 + [4] * 2, dtype=np.int32)
    M = 40
    o1, f1 = orc.sorted_f_exact(s, o, M, orc.DP)
    o2, f2 = orc.sorted_f_prefix(s, o, M)
    assert f1.tolist() == f2.tolist()
    assert orc.list_schedule_alg1(s, o, M, o1)[1] == orc.list_schedule_alg1(s, o, M, o2)[1]


# ----------------------------------------------------------------------------- optimum and the 48x bound
def test_bruteforce_and_approximation_bound(golden):
    rng = np.random.default_rng(2024)
    for trial in range(25):
        n = int(rng.integers(2, 7))
        M = int(rng.integers(10, 40))
        s, o = random_instance(rng, n, M, M // 2, 6)
        best_list, best_order = orc.bruteforce_best_order(s, o, M)
        opt, p = orc.bruteforce_opt(s, o, M, best_list + 1)
        assert 0 < opt <= best_list                        # list schedules are feasible schedules
        assert orc.check_schedule(s, o, M, p)["feasible"] and orc.check_schedule(s, o, M, p)["tel"] == opt
        assert opt >= int(o.sum())                         # nobody finishes before decoding o_i tokens
        for solver in (orc.ENUM_ALG1, orc.ENUM_SUM, orc.DP):
            order, _ = orc.sorted_f_exact(s, o, M, solver)
            tel = orc.list_schedule_alg1(s, o, M, order)[1]
            assert best_list <= tel < golden["approx_ratio_bound"] * opt
        order, _ = orc.sorted_f_prefix(s, o, M)
        assert orc.list_schedule_alg1(s, o, M, order)[1] >= best_list


def test_bruteforce_on_first_eight_of_tiny_backlog():
    inst = W.tiny()
    s, o = inst.s[:8], inst.o[:8]
    best_list, _ = orc.bruteforce_best_order(s, o, inst.M)
    opt, p = orc.bruteforce_opt(s, o, inst.M, best_list + 1)
    assert opt <= best_list and orc.check_schedule(s, o, inst.M, p)["feasible"]
    order, _ = orc.sorted_f_exact(s, o, inst.M, orc.DP)
    assert best_list <= orc.list_schedule_alg1(s, o, inst.M, order)[1] < 48 * opt


# ----------------------------------------------------------------------------- moves and local search
def test_move_codes_enumerate_the_neighbourhood():
    for n in (2, 3, 7, 16):
        nsw = n * (n - 1) // 2
        swaps = [orc.decode_move(n, c) for c in range(nsw)]
        assert [(i, j) for _, i, j in swaps] == list(itertools.combinations(range(n), 2))
        assert all(t == 0 for t, _, _ in swaps)
        ins = [orc.decode_move(n, c) for c in range(nsw, nsw + n * (n - 1))]
        assert [(i, j) for _, i, j in ins] == [(i, j) for i in range(n) for j in range(n) if i != j]
        assert all(t == 1 for t, _, _ in ins)
        with pytest.raises(ValueError):
            orc.decode_move(n, nsw + n * (n - 1))
        base = np.arange(n, dtype=np.int32)[::-1].copy()
        for t, i, j in swaps + ins:
            ref = base.tolist()
            if t == 0:
                ref[i], ref[j] = ref[j], ref[i]
            else:
                x = ref.pop(i)
                ref.insert(j, x)
            assert orc.apply_move(base, t, i, j).tolist() == ref
            if t == 1:
                assert ref[j] == base[i]                   # the moved request lands at position j


def test_sampled_moves_are_valid_and_reproducible():
    n = 50
    seen = set()
    for m in range(2000):
        t, i, j = orc.sample_move(n, 42, 3, m)
        assert t in (0, 1) and 0 <= i < n and 0 <= j < n and i != j
        if t == 0:
            assert i < j
        assert (t, i, j) == orc.sample_move(n, 42, 3, m)
        seen.add((t, i, j))
    assert len(seen) > 1500                                # spread over the neighbourhood
    assert orc.sample_move(n, 42, 4, 0) != orc.sample_move(n, 42, 3, 0) or orc.sample_move(n, 42, 4, 1) != orc.sample_move(n, 42, 3, 1)


def test_local_search_descends_to_a_local_optimum():
    rng = np.random.default_rng(31)
    for trial in range(8):
        n = int(rng.integers(4, 9))
        M = int(rng.integers(14, 40))
        s, o = random_instance(rng, n, M, M // 2, 6)
        start = rng.permutation(n).astype(np.int32)
        t0 = orc.list_schedule_alg1(s, o, M, start)[1]
        for nb in (orc.SWAP, orc.SWAP_INSERT):
            order, tel, done, trace = orc.local_search(s, o, M, nb, 100, start)
            assert sorted(order.tolist()) == list(range(n))
            assert tel == orc.list_schedule_alg1(s, o, M, order)[1] <= t0
            accepted = [int(t) for _, t in trace[:-1]]
            assert accepted == sorted(accepted, reverse=True) and len(set(accepted)) == len(accepted)
            assert all(t < t0 for t in accepted)
            # every neighbour of the result is no better (recomputed with the literal executor)
            ncodes = n * (n - 1) // 2 + (n * (n - 1) if nb == orc.SWAP_INSERT else 0)
            for c in range(ncodes):
                cand = orc.apply_move(order, *orc.decode_move(n, c))
                assert orc.list_schedule_alg1(s, o, M, cand)[1] >= tel
            assert tel >= orc.bruteforce_best_order(s, o, M)[0]


def test_local_search_picks_lowest_code_among_equal_best():
    # all requests identical: every neighbour ties with the start, nothing is accepted
    s, o = np.full(6, 3, dtype=np.int32), np.full(6, 2, dtype=np.int32)
    order, tel, done, trace = orc.local_search(s, o, 11, orc.SWAP_INSERT, 10, np.arange(6))
    assert done == 1 and trace[0][0] == 0 and order.tolist() == list(range(6))


# ----------------------------------------------------------------------------- workloads
def test_workloads_are_deterministic_and_shaped():
    a, b = W.mixed_1k(), W.mixed_1k()
    assert (a.s == b.s).all() and (a.o == b.o).all() and a.checksum() == b.checksum()
    assert a.checksum() != W.mixed_1k(seed=11).checksum()
    big = W.mixed_10k()
    assert big.n == 10000 and big.M == 262144
    docs = big.s >= 4096
    assert 0.17 < docs.mean() < 0.23
    assert big.s[~docs].max() <= 2048 and big.s[~docs].min() >= 16
    assert big.o[~docs].max() <= 1024 and big.o[~docs].min() >= 8
    assert big.o[docs].min() >= 128 and big.o[docs].max() <= 512
    assert (big.s.astype(np.int64) + big.o).sum() > 20 * big.M          # overloaded regime
    t = W.tiny()
    assert t.n == 16 and t.s.min() >= 1 and t.s.max() <= 32 and t.o.min() >= 1 and t.o.max() <= 32


# ----------------------------------------------------------------------------- Algorithm 3 (Local Swap Search)
def test_local_swap_worked_by_hand():
    # A(1,5) B(2,5) C(5,3) D(8,1) E(9,1); sizes 6,7,8,9,10; M = 14.
    # First fit: A, B (mem 13).  out=A: C,D,E all overflow.  out=B: C fits exactly (14) and has the
    # smaller o -> X = [A, C].  Restart: nothing outside is both smaller in o and fits -> stop.
    s, o = np.array([1, 2, 5, 8, 9], dtype=np.int32), np.array([5, 5, 3, 1, 1], dtype=np.int32)
    X, swaps = orc.local_swap_batch(np.arange(5), s, o, 14)
    assert X.tolist() == [0, 2] and swaps == 1
    # equal sizes: the walk is out-major, in-minor and restarts after every swap.
    # P(4,6) Q(4,6) R(6,4) S(8,2), all of size 10, M = 20: P->R, then R->S, then Q->R.
    s, o = np.array([4, 4, 6, 8], dtype=np.int32), np.array([6, 6, 4, 2], dtype=np.int32)
    X, swaps = orc.local_swap_batch(np.arange(4), s, o, 20)
    assert X.tolist() == [3, 2] and swaps == 3


def test_local_swap_example1_and_properties(golden):
    s = np.array([63] + [1] * 21, dtype=np.int32)
    o = np.array([1] + [2] * 21, dtype=np.int32)
    order, offs, swaps = orc.sorted_f_local_swap(s, o, golden["example1_M"])
    assert offs.tolist() == [0, 21, 22] and order[-1] == 0 and swaps == 0
    assert orc.list_schedule_alg1(s, o, 64, order)[1] == golden["example1_tel_sortedf"]
    rng = np.random.default_rng(404)
    for trial in range(150):
        n = int(rng.integers(1, 40))
        M = int(rng.integers(10, 120))
        s, o = random_instance(rng, n, M, M // 2, M // 2)
        ids = np.arange(n)
        X, swaps = orc.local_swap_batch(ids, s, o, M)
        T = s.astype(np.int64) + o
        mem = int(T[X].sum())
        assert len(set(X.tolist())) == len(X) and mem <= M
        # the batch size is the first-fit size: the longest prefix by ascending s+o that fits
        by_size = sorted(range(n), key=lambda i: (T[i], i))
        k0, acc = 0, 0
        for i in by_size:
            if acc + T[i] <= M:
                acc += T[i]; k0 += 1
        assert len(X) == k0
        # local optimum by the definition of Section 5.2: no swap keeps memory and lowers F
        outside = [i for i in range(n) if i not in set(X.tolist())]
        for a in X:
            for b in outside:
                assert not (mem + T[b] - T[a] <= M and o[b] < o[a])
        # never worse than where it started
        assert int(o[X].sum()) <= int(o[by_size[:k0]].sum())
        assert (swaps == 0) == (sorted(X.tolist()) == sorted(by_size[:k0]))
        order, offs, _ = orc.sorted_f_local_swap(s, o, M)
        assert sorted(order.tolist()) == list(range(n)) and offs[0] == 0 and offs[-1] == n
        for a, b in zip(offs[:-1], offs[1:]):
            assert (np.diff(o[order[a:b]]) >= 0).all() and int(T[order[a:b]].sum()) <= M
        assert order[:offs[1]].tolist() == sorted(X.tolist(), key=lambda i: (o[i], i))


# ----------------------------------------------------------------------------- Sorted-G (prefill-weighted metric)
def test_sorted_g_reduces_to_f_and_differs_by_hand():
    from fractions import Fraction
    rng = np.random.default_rng(606)
    for trial in range(60):
        n = int(rng.integers(1, 60))
        M = int(rng.integers(10, 300))
        s, o = random_instance(rng, n, M, M // 2, M // 3 + 1)
        # alpha = 0 recovers the F-metric (Section 7), whatever the denominator
        for den in (1, 7):
            og, fg = orc.sorted_g_prefix(s, o, M, 0, den)
            of, ff = orc.sorted_f_prefix(s, o, M)
            assert (og == of).all() and (fg == ff).all()
            og, fg = orc.sorted_g_local_swap(s, o, M, 0, den)
            ol, fl, _ = orc.sorted_f_local_swap(s, o, M)
            assert (og == ol).all() and (fg == fl).all()
        # first batch against the definition with exact fractions: G(X) = sum(alpha*s+o)/|X|^2
        a_num, a_den = int(rng.integers(0, 6)), int(rng.integers(1, 5))
        alpha = Fraction(a_num, a_den)
        order, offs = orc.sorted_g_prefix(s, o, M, a_num, a_den)
        by_size = sorted(range(n), key=lambda i: (int(s[i]) + int(o[i]), int(o[i]), i))
        best, best_k, mem, tot = None, 0, 0, Fraction(0)
        for k, i in enumerate(by_size, 1):
            mem += int(s[i]) + int(o[i])
            if mem > M:
                break
            tot += alpha * int(s[i]) + int(o[i])
            g = tot / (k * k)
            if best is None or g < best or (g == best and k > best_k):
                best, best_k = g, k
        assert offs[1] == best_k and sorted(order[:best_k].tolist()) == sorted(by_size[:best_k])
    # by hand: B(1,4) B(1,4) A(30,1), M = 41.  F: 4/1, 8/4, 9/9 -> all three.  alpha = 1: 5/1, 10/4,
    # 41/9 -> only the two small prompts.
    s, o = np.array([30, 1, 1], dtype=np.int32), np.array([1, 4, 4], dtype=np.int32)
    assert orc.sorted_g_prefix(s, o, 41, 0, 1)[1].tolist() == [0, 3]
    assert orc.sorted_g_prefix(s, o, 41, 1, 1)[1].tolist() == [0, 2, 3]
    # Algorithm 3 under G: swapping in the long prompt A(30,1) for B lowers sum(o) but not sum(s+o)
    s, o = np.array([1, 1, 3], dtype=np.int32), np.array([4, 4, 1], dtype=np.int32)      # sizes 5, 5, 4; M = 9
    assert sorted(orc.sorted_f_local_swap(s, o, 9)[0][:2].tolist()) == [0, 2]            # first fit {2,0}; nothing better
    s, o = np.array([1, 1, 4], dtype=np.int32), np.array([4, 4, 1], dtype=np.int32)      # sizes 5, 5, 5; M = 10
    assert sorted(orc.sorted_f_local_swap(s, o, 10)[0][:2].tolist()) == [1, 2]           # F: o 1 < 4 -> swap request 0 out
    assert sorted(orc.sorted_g_local_swap(s, o, 10, 1, 1)[0][:2].tolist()) == [0, 1]     # G, alpha=1: weights 5,5,5 -> no swap


# ---------------------------------------------------------------------------------------------
# Algorithm 4 (Quantile Greedy Selection)
# ---------------------------------------------------------------------------------------------
def test_mix64_is_splitmix64():
    # first three outputs of splitmix64 seeded with 0 (Steele, Lea, Flood; the generator's
    # published reference values); mix64(z) is one step from state z
    gamma = 0x9E3779B97F4A7C15
    assert orc.mix64(0) == 0xE220A8397B1DCDAF
    assert orc.mix64(gamma) == 0x6E789E6AA1B965F4
    assert orc.mix64(2 * gamma) == 0x06C45D188009454F


def test_quantile_greedy_worked_by_hand():
    s = np.array([3, 5, 2, 8, 1, 4])
    o = np.array([2, 1, 4, 3, 5, 2])
    ids = np.arange(6)
    # I by (o, index): 1, 0, 5, 3, 2, 4.  Sample {0,1,2}: s+o = 5,6,6 -> Q_p = 5 (position
    # floor(0.3*2) = 0); o = 1,2,4 -> Q_o = 1.  Nothing passes both thresholds (request 1 has
    # s+o = 6).  Ratios o/(s+o): r1 1/6, r3 3/11, r5 2/6, r0 2/5, r2 4/6, r4 5/6 -> first fit at
    # M = 20 takes r1 (6), r3 (17) and nothing else.
    X, qp, qo = orc.quantile_greedy_batch(ids, s, o, 20, [0, 1, 2])
    assert (qp, qo) == (5, 1) and X.tolist() == [1, 3]
    # Sample {0,1,3,5,2}: s+o = 5,6,6,6,11 -> Q_p = 6 (position floor(0.3*4) = 1); o = 1,2,2,3,4
    # -> Q_o = 2.  Pass 1 admits r1, r0, r5 (mem 17).  Left over by ratio: r3, r2, r4.
    X, qp, qo = orc.quantile_greedy_batch(ids, s, o, 18, [0, 1, 3, 5, 2])
    assert (qp, qo) == (6, 2) and X.tolist() == [1, 0, 5]
    # M = 23: pass 2 skips r3 (28 > 23) and goes on to admit r2 (23), then r4 no longer fits.
    X, _, _ = orc.quantile_greedy_batch(ids, s, o, 23, [0, 1, 3, 5, 2])
    assert X.tolist() == [1, 0, 5, 2]
    # M = 15: r5 passes both thresholds but does not fit after r1 and r0; it falls to pass 2.
    X, _, _ = orc.quantile_greedy_batch(ids, s, o, 15, [0, 1, 3, 5, 2])
    assert X.tolist() == [1, 0]
    # equal ratios (1/2 for both) keep the order of I; 1/3 < 333334/1000001 is decided exactly
    # (thresholds (2, 1) from the sample {r2}: pass 1 takes r2 only; r1 then fills M = 10, r0 misfits)
    X, _, _ = orc.quantile_greedy_batch([0, 1, 2], [4, 2, 1], [4, 2, 1], 10, [2])
    assert X.tolist() == [2, 1]
    # exact ratio comparison: with k = 2^28, r0 = (s k-1, o k) has ratio k/(2k-1) and r1 = (s k, o k+1)
    # has (k+1)/(2k+1), smaller by 1/((2k-1)(2k+1)) ~ 2^-58 -- equal in double precision.  Pass 1
    # takes r2 (thresholds (10, 1) from the sample {r2}); pass 2 must try r1 first, which then
    # fills M = 10 + 2k+1 so that r0 misfits (a floating-point tie would admit r0 instead).
    k = 1 << 28
    X, _, _ = orc.quantile_greedy_batch([0, 1, 2], [k - 1, k, 9], [k, k + 1, 1], 10 + 2 * k + 1, [2])
    assert X.tolist() == [2, 1]


def test_quantile_greedy_properties():
    rng = np.random.default_rng(77)
    for trial in range(40):
        n = int(rng.integers(1, 60))
        M = int(rng.integers(20, 200))
        s, o = random_instance(rng, n, M, M // 2, max(2, M // 4))
        T = s + o
        ids = rng.permutation(n)[: int(rng.integers(1, n + 1))]
        sample = orc.quantile_sample(ids, o, 1234 + trial, trial)
        m = len(ids)
        assert len(sample) == max(1, m // 2) and len(set(sample.tolist())) == len(sample)
        assert set(sample.tolist()) <= set(ids.tolist())
        assert sample.tolist() == orc.quantile_sample(ids, o, 1234 + trial, trial).tolist()
        X, qp, qo = orc.quantile_greedy_batch(ids, s, o, M, sample)
        # thresholds against numpy's own lower quantile (element at floor(0.3 (m-1)))
        if (3 * (len(sample) - 1)) % 10 != 0:        # away from the points where 0.3*(m-1) rounds in floating point
            assert qp == int(np.quantile(T[sample], 0.3, method="lower"))
            assert qo == int(np.quantile(o[sample], 0.3, method="lower"))
        assert len(set(X.tolist())) == len(X) >= 1 and set(X.tolist()) <= set(ids.tolist())
        mem = int(T[X].sum())
        assert mem <= M
        rest = [r for r in ids.tolist() if r not in set(X.tolist())]
        assert all(mem + T[r] > M for r in rest)                 # first fit over everything: X is maximal
        # the members that pass both thresholds come first, in ascending (o, index)
        core = [r for r in X.tolist() if T[r] <= qp and o[r] <= qo]
        k = 0
        while k < len(X) and T[X[k]] <= qp and o[X[k]] <= qo:
            k += 1
        head = X[:k].tolist()
        assert head == sorted(head, key=lambda r: (o[r], r))
        # every request that passes both thresholds and is NOT in the head was refused for memory
        # at its turn: the head members before it already fill M - T[r]
        I = sorted(ids.tolist(), key=lambda r: (o[r], r))
        mem1 = 0
        for r in I:
            if T[r] <= qp and o[r] <= qo:
                if mem1 + T[r] <= M:
                    assert r in head
                    mem1 += T[r]
        del core


def test_quantile_sample_varies_with_seed_and_batch():
    o = np.arange(1, 41)
    ids = np.arange(40)
    a = orc.quantile_sample(ids, o, 1, 0).tolist()
    assert a != orc.quantile_sample(ids, o, 2, 0).tolist()
    assert a != orc.quantile_sample(ids, o, 1, 1).tolist()
    # the sample is the half with the smallest keys mix(seed ^ mix(batch * 2^32 + id))
    keys = {i: orc.mix64(1 ^ orc.mix64((0 << 32) + i)) for i in range(40)}
    assert sorted(a) == sorted(sorted(range(40), key=lambda i: keys[i])[:20])
    # about half of all requests over many seeds: no request is favoured
    hits = np.zeros(40)
    for seed in range(400):
        hits[orc.quantile_sample(ids, o, seed, 0)] += 1
    assert hits.min() > 140 and hits.max() < 260


def test_sorted_f_quantile_is_a_partition_into_feasible_maximal_batches():
    rng = np.random.default_rng(78)
    for trial in range(20):
        n = int(rng.integers(1, 80))
        M = int(rng.integers(20, 300))
        s, o = random_instance(rng, n, M, M // 2, max(2, M // 4))
        T = s + o
        order, offs = orc.sorted_f_quantile(s, o, M, 99)
        assert sorted(order.tolist()) == list(range(n))
        assert offs[0] == 0 and offs[-1] == n and np.all(np.diff(offs) >= 1)
        left = set(range(n))
        for b in range(len(offs) - 1):
            X = order[offs[b]: offs[b + 1]].tolist()
            assert X == sorted(X, key=lambda r: (o[r], r))
            mem = int(T[X].sum())
            assert mem <= M
            left -= set(X)
            assert all(mem + T[r] > M for r in left)
            # the batch is what the one-batch routine returns on the requests still there
            rem = sorted(left | set(X))
            sample = orc.quantile_sample(rem, o, 99, b)
            Xb, _, _ = orc.quantile_greedy_batch(rem, s, o, M, sample)
            assert sorted(Xb.tolist()) == sorted(X)
    # Example 1 (Section 3): one request (s=63, o=1) and 21 requests (s=1, o=2), M = 64
    s = np.array([63] + [1] * 21); o = np.array([1] + [2] * 21)
    order, offs = orc.sorted_f_quantile(s, o, 64, 5)
    tel = orc.list_schedule_alg1(s, o, 64, order)[1]
    assert tel in (45, 64)                                     # one of the two batch orders the example discusses


# ---------------------------------------------------------------------------------------------
# Online arrivals (Section 6.2, Section 7's Poisson experiment)
# ---------------------------------------------------------------------------------------------
ONLINE_POLICIES = (orc.FCFS, orc.SOF, orc.SORTED_F)


def test_online_with_everything_present_at_time_zero_is_the_offline_model():
    rng = np.random.default_rng(91)
    for trial in range(12):
        n = int(rng.integers(1, 40))
        M = int(rng.integers(20, 200))
        s, o = random_instance(rng, n, M, M // 2, max(2, M // 4))
        a = np.zeros(n, dtype=np.int32)
        for pol in (orc.FCFS, orc.SOF):
            p, tot = orc.online_schedule(a, s, o, M, pol)
            rp, rtel, _ = orc.list_schedule_alg1(s, o, M, orc.policy_order(s, o, pol))
            assert (p == rp).all() and tot == rtel
        # one planning pass over the whole backlog, never repeated: Sorted-F with Algorithm 3
        p, tot = orc.online_schedule(a, s, o, M, orc.SORTED_F, period=1 << 30, lookahead=n)
        order = orc.sorted_f_local_swap(s, o, M)[0]
        rp, rtel, _ = orc.list_schedule_alg1(s, o, M, order)
        assert (p == rp).all() and tot == rtel


def test_online_underloaded_requests_start_on_arrival():
    rng = np.random.default_rng(92)
    n, M = 30, 100
    s, o = random_instance(rng, n, M, 50, 20)
    a = np.cumsum(rng.integers(21, 40, n)).astype(np.int32)        # gaps longer than any decode
    for pol in ONLINE_POLICIES:
        p, tot = orc.online_schedule(a, s, o, M, pol)
        assert (p == a).all() and tot == int(o.sum())


def test_online_schedules_are_feasible_and_fcfs_is_earliest_fit_in_arrival_order():
    rng = np.random.default_rng(93)
    for trial in range(10):
        n = int(rng.integers(2, 50))
        M = int(rng.integers(20, 120))
        s, o = random_instance(rng, n, M, M // 2, max(2, M // 4))
        a = np.sort(rng.integers(0, 3 * n, n)).astype(np.int32)
        for pol in ONLINE_POLICIES:
            p, tot = orc.online_schedule(a, s, o, M, pol, period=int(rng.integers(1, 6)), lookahead=int(rng.integers(1, 12)))
            assert (p >= a).all()
            chk = orc.check_schedule(s, o, M, p)
            assert chk["feasible"] and chk["peak"] <= M and tot == chk["tel"] - int(a.sum())
        # FCFS by its definition: request i starts at the first p >= max(a_i, p_{i-1}) at which
        # every round of its stay is within M, given the earlier requests
        p, _ = orc.online_schedule(a, s, o, M, orc.FCFS)
        U = np.zeros(int(a.max()) + int(o.sum()) + 2, dtype=np.int64)
        prev = 0
        for i in range(n):
            q = max(int(a[i]), prev)
            while any(U[q + j] + s[i] + j > M for j in range(1, o[i] + 1)):
                q += 1
            assert p[i] == q
            for j in range(1, o[i] + 1):
                U[q + j] += s[i] + j
            prev = q


def test_online_fcfs_and_shortest_first_worked_by_hand():
    # M = 10; r0 (a 0, s 4, o 3), r1 (a 0, s 5, o 4), r2 (a 1, s 2, o 1).
    a, s, o = [0, 0, 1], [4, 5, 2], [3, 4, 1]
    # FCFS: iteration 1 admits r0 (rounds 1-3 use 5,6,7); r1 would make round 1 use 11.  r1 stays
    # at the head and is refused in iterations 2 and 3 (rounds 2, 3 still hold 6, 7), which also
    # holds r2 back; iteration 4 admits r1 (p = 3) and then r2 (round 4: 6 + 3 = 9).
    p, tot = orc.online_schedule(a, s, o, 10, orc.FCFS)
    assert p.tolist() == [0, 3, 3] and tot == 3 + 7 + 3
    # shortest first: in iteration 2 r2 (o = 1) goes ahead of r1 and fits (round 2: 6 + 3 = 9).
    p, tot = orc.online_schedule(a, s, o, 10, orc.SOF)
    assert p.tolist() == [0, 3, 1] and tot == 3 + 7 + 1


def test_sorted_f_online_worked_by_hand():
    M = 10
    # Example A (period 3, look-ahead 2): r0, r1 = (a 0, s 1, o 2), r2 = (0, 6, 1), r3 = (1, 1, 1),
    # r4 = (2, 2, 1), r5 = (6, 3, 2).
    #  it 1: first plan.  By (s+o, index): r0, r1 | r2 -- only the first two are planned: one batch
    #        {r0, r1}; list r0, r1, r2.  r0, r1 start (round 1 holds 4, round 2 holds 6); r2 would
    #        make round 1 hold 11.
    #  it 2: r3 arrives, goes to the tail (1 arrival < half of 3).  r2 refused (round 2: 6 + 7);
    #        r3 waits behind it.
    #  it 3: r4 arrives: 2 arrivals >= half of 3 -> new plan: r3, r4 | r2 -> list r3, r4, r2.
    #        r3 and r4 start (round 3 holds 5); r2 refused (12).
    #  it 4: r2 starts.  it 7: r5 has arrived, the list had run empty -> plan; r5 starts.
    a, s, o = [0, 0, 0, 1, 2, 6], [1, 1, 6, 1, 2, 3], [2, 2, 1, 1, 1, 2]
    p, tot = orc.online_schedule(a, s, o, M, orc.SORTED_F, period=3, lookahead=2)
    assert p.tolist() == [0, 0, 3, 2, 2, 6] and tot == 2 + 2 + 4 + 2 + 1 + 2
    # with a look-ahead of 3 the first plan swaps r0 out for r2 (o 1 < 2, memory 3+7 = 10 fits):
    # batch {r2, r1}, then {r0}
    p3, _ = orc.online_schedule(a, s, o, M, orc.SORTED_F, period=3, lookahead=3)
    assert p3[2] == 0 and p3[1] == 0 and p3[0] > 0
    # Example B (look-ahead 10): r0 = (0, 5, 4), r1 = (0, 6, 3), r2 = (0, 6, 2), r3 = (0, 7, 2),
    # r4 = (1, 1, 1).  First plan: batches {r2}, {r3}, {r1}, {r0} (each is alone: two never fit;
    # Algorithm 3 walks to the shortest decode).  r2 starts in iteration 1; r3 is refused in
    # iterations 1 and 2 (rounds 1, 2 hold 7, 8); r4 arrives in iteration 2 and waits at the tail
    # although it would fit (8 + 2).
    a, s, o = [0, 0, 0, 0, 1], [5, 6, 6, 7, 1], [4, 3, 2, 2, 1]
    #  period 2: iteration 3 plans again: by size r4 first -> list r4, r3, r1, r0; r4 and r3 start
    #  (round 3: 2 + 8 = 10), r1 in iteration 5, r0 in iteration 8.
    p, tot = orc.online_schedule(a, s, o, M, orc.SORTED_F, period=2, lookahead=10)
    assert p.tolist() == [7, 4, 0, 2, 2] and tot == 11 + 7 + 2 + 4 + 2
    #  period 100: no new plan (1 arrival < half of 4): r4 stays last and starts with r0 in iteration 8.
    p, _ = orc.online_schedule(a, s, o, M, orc.SORTED_F, period=100, lookahead=10)
    assert p.tolist() == [7, 4, 0, 2, 7]


def test_online_overload_ranking_of_the_three_policies():
    # Section 7, online experiment: under overload Sorted-F-Online has the lowest mean latency and
    # FCFS by far the highest (the paper: 15-40 % below shortest-decode-first, 83-88 % below FCFS)
    inst = W.online_poisson(0.25, horizon=1500, seed=3)
    lat = {pol: orc.online_schedule(inst.a, inst.s, inst.o, inst.M, pol)[1] for pol in ONLINE_POLICIES}
    assert lat[orc.SORTED_F] < lat[orc.SOF] < lat[orc.FCFS]
    assert lat[orc.SORTED_F] < 0.5 * lat[orc.FCFS]


# ---------------------------------------------------------------------------------------------
# Sorted-F + A_min (Section 5.5, Algorithm 5): executor under lower-bound predictions
# ---------------------------------------------------------------------------------------------
def test_amin_with_exact_predictions_is_algorithm_1():
    rng = np.random.default_rng(101)
    for trial in range(15):
        n = int(rng.integers(1, 40))
        M = int(rng.integers(20, 200))
        s, o = random_instance(rng, n, M, M // 2, max(2, M // 4))
        order = rng.permutation(n).astype(np.int32)
        p, tel, ev, peak = orc.amin_schedule(s, o, o, M, order)
        rp, rtel, _ = orc.list_schedule_alg1(s, o, M, order)
        assert (p == rp).all() and tel == rtel and ev == 0
        assert peak == orc.check_schedule(s, o, M, rp)["peak"]


def test_amin_never_exceeds_memory_and_finishes_everything():
    rng = np.random.default_rng(102)
    total_ev = 0
    for trial in range(25):
        n = int(rng.integers(2, 50))
        M = int(rng.integers(30, 200))
        s, o = random_instance(rng, n, M, M // 2, max(2, M // 3))
        lower = np.maximum(1, np.floor(o * rng.uniform(0.1, 1.0, n))).astype(np.int32)
        order = rng.permutation(n).astype(np.int32)
        p, tel, ev, peak = orc.amin_schedule(s, lower, o, M, order)
        total_ev += ev
        assert peak <= M and (p >= 0).all() and tel == int((p + o).sum())
        # the final runs alone (evicted attempts also used memory, so this is a lower bound on
        # the peak) are a feasible schedule in the sense of the integer program
        chk = orc.check_schedule(s, o, M, p)
        assert chk["feasible"] and chk["peak"] <= peak
    assert total_ev > 20                                # the eviction path really ran


def test_amin_worked_by_hand():
    # M = 8, list r0, r1.  r0 = (s 2, l 2, o 4), r1 = (s 3, l 1, o 2).
    #  it 1: both start (projected round 1: 3 + 4).  it 2: both are in their 2nd round, estimates
    #  2 and 2, round 2 would hold 4 + 5 = 9 > 8: equal estimates, the lower index r0 is evicted.
    #  it 3: r1 has finished (c = 2); r0 starts again (p = 2) and runs 4 rounds: c = 6.
    p, tel, ev, peak = orc.amin_schedule([2, 3], [2, 1], [4, 2], 8, [0, 1])
    assert p.tolist() == [2, 0] and tel == 6 + 2 and ev == 1 and peak == 7
    # r0 = (s 2, l 3, o 4), r1 = (s 3, l 1, o 3).
    #  it 2: estimates 3 and 2, round 2 would hold 9: r1 (smaller estimate) is evicted, keeps 2.
    #  it 3, 4: r1 refused (round 3: 5 + 4, round 4: 6 + 4).  it 5: r0 is done (c = 4), r1 starts
    #  (p = 4), c = 7.
    p, tel, ev, peak = orc.amin_schedule([2, 3], [3, 1], [4, 3], 8, [0, 1])
    assert p.tolist() == [0, 4] and tel == 4 + 7 and ev == 1 and peak == 7
    # an evicted request goes back IN FRONT of requests that never started: r2 = (s 1, l 1, o 1)
    # is behind r1 in the list and must wait for it although it would fit in iteration 3
    p, tel, ev, _ = orc.amin_schedule([2, 3, 1], [3, 1, 1], [4, 3, 1], 8, [0, 1, 2])
    assert p.tolist() == [0, 4, 4] and ev == 1


def test_amin_per_round_form_equals_the_set_form():
    """O14' (projected memory kept per round) against O14 (projection re-derived from the sets):
    start times, TEL, evictions and peak, over tight and loose memories and crude lower bounds."""
    rng = np.random.default_rng(103)
    evs = 0
    for trial in range(300):
        n = int(rng.integers(1, 45))
        M = int(rng.integers(12, 160))
        s, o = random_instance(rng, n, M, max(1, M // 2), max(2, M // int(rng.integers(2, 6))))
        frac = rng.uniform(0.0, 1.0) if trial % 3 else 0.0
        lower = np.clip(np.floor(o * rng.uniform(frac, 1.0, n)), 1, o).astype(np.int32)
        order = rng.permutation(n).astype(np.int32)
        a = orc.amin_schedule(s, lower, o, M, order)
        b = orc.amin_schedule_rounds(s, lower, o, M, order)
        assert (a[0] == b[0]).all() and a[1:] == b[1:], trial
        evs += a[2]
    assert evs > 300
    # the worked cases
    assert orc.amin_schedule_rounds([2, 3], [2, 1], [4, 2], 8, [0, 1])[0].tolist() == [2, 0]
    assert orc.amin_schedule_rounds([2, 3, 1], [3, 1, 1], [4, 3, 1], 8, [0, 1, 2])[0].tolist() == [0, 4, 4]
