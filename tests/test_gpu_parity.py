"""GPU parity: every integer the CUDA library returns equals the CPU oracle's on the same inputs.

All calls go through the C-ABI (``binding.Scheduler`` only marshals arguments).  Bit-exact: TELs,
start times, feasibility flags, Sorted-F orders and batch boundaries, local-search traces.
"""
import numpy as np
import pytest

import oracle as orc
from paper_2508_06133_b200 import binding as kv
from paper_2508_06133_b200 import workloads as W

pytestmark = pytest.mark.gpu


def rand_instance(rng, n, M, smax, omax):
    s = rng.integers(1, smax + 1, n).astype(np.int32)
    o = rng.integers(1, omax + 1, n).astype(np.int32)
    bad = s.astype(np.int64) + o > M
    s[bad] = 1
    return s, o


def all_codes(n, inserts=True):
    return np.arange(n * (n - 1) // 2 + (n * (n - 1) if inserts else 0), dtype=np.int64)


def oracle_moves(s, o, M, base, codes):
    mv = [orc.decode_move(len(s), int(c)) for c in codes]
    return orc.eval_moves(s, o, M, base, [m[0] for m in mv], [m[1] for m in mv], [m[2] for m in mv])


# ------------------------------------------------------------------------------------ ORDER
def test_orders_small_random_instances_tel_and_starts():
    rng = np.random.default_rng(1)
    for trial in range(60):
        n = int(rng.integers(1, 70))
        M = int(rng.integers(8, 300))
        s, o = rand_instance(rng, n, M, max(1, M // 2), max(1, M // 3))
        orders = np.stack([rng.permutation(n) for _ in range(9)]).astype(np.int32)
        with kv.Scheduler(s, o, M) as h:
            tel, feas, starts = h.eval_batch(kv.CAND_ORDER, orders, want_feasible=True, want_starts=True)
        assert feas.all()
        for c in range(len(orders)):
            p, t, _ = orc.list_schedule_alg1(s, o, M, orders[c])
            assert tel[c] == t
            assert (starts[c] == p).all()


def test_orders_paper_example_and_closed_form(golden):
    s = np.array([63] + [1] * 21, dtype=np.int32)
    o = np.array([1] + [2] * 21, dtype=np.int32)
    orders = np.stack([np.arange(22), np.array(list(range(1, 22)) + [0])]).astype(np.int32)
    with kv.Scheduler(s, o, 64) as h:
        tel, _, _ = h.eval_batch(kv.CAND_ORDER, orders)
    assert tel.tolist() == [golden["example1_tel_mcsf"], golden["example1_tel_sortedf"]]
    M = 6561
    s = np.array([80] * M + [1] * 59049, dtype=np.int32)
    o = np.array([1] * M + [2] * 59049, dtype=np.int32)
    with kv.Scheduler(s, o, M) as h:
        tel, _, _ = h.eval_batch(kv.CAND_ORDER, np.arange(len(s), dtype=np.int32)[None, :])
    assert tel[0] == golden["thm1_M6561_tel_mcsf"]


def test_orders_long_waits_and_ring_wrap():
    """Few huge requests force waits longer than a decode length; tiny o_max wraps the ring often."""
    rng = np.random.default_rng(2)
    for omax, M in ((1, 50), (2, 40), (3, 64), (40, 100), (200, 1000)):
        n = 120
        s = rng.integers(1, M - omax, n).astype(np.int32)
        o = rng.integers(1, omax + 1, n).astype(np.int32)
        s[::7] = M - o[::7]                                  # requests that need the machine alone
        orders = np.stack([rng.permutation(n) for _ in range(5)]).astype(np.int32)
        with kv.Scheduler(s, o, M) as h:
            tel, _, starts = h.eval_batch(kv.CAND_ORDER, orders, want_starts=True)
        for c in range(5):
            p, t, _ = orc.list_schedule_rounds(s, o, M, orders[c])
            assert tel[c] == t and (starts[c] == p).all()


@pytest.mark.parametrize("sim", ["", "smem", "hybrid"])
def test_orders_wait_decided_behind_the_first_chunk(sim, monkeypatch):
    """The simulators look at the first 32 rounds of a window before anything else.  Here the only
    rounds over budget lie behind them: with M = 195, A = (s 100, o 40) runs from round 0 and peaks at
    140 tokens in round 39; B = (s 20, o 60) fits beside it in rounds 0..31 (at most 132 + 52 = 184)
    and first overflows in round 37 (138 + 58 = 196), so its wait comes from the second chunk alone.
    Also with the pair shifted to every kind of start offset inside a chunk, with longer tails, and
    in other orders; on the default simulator and on the two with shared-memory timelines."""
    if sim:
        monkeypatch.setenv("KVSCHED_SIM", sim)
    M = 195
    for lead in (0, 1, 5, 17, 31, 32, 33, 63):                     # a request of `lead` rounds in front moves t
        for tail in (60, 90, 150):
            s = np.array([50, 100, 20, 3, 7], dtype=np.int32)
            o = np.array([max(lead, 1), 40, tail, 64, 33], dtype=np.int32)
            n = len(s)
            orders = np.stack([np.arange(n), np.arange(n)[::-1], np.roll(np.arange(n), 1)]).astype(np.int32)
            with kv.Scheduler(s, o, M) as h:
                tel, _, starts = h.eval_batch(kv.CAND_ORDER, orders, want_starts=True)
            for c in range(len(orders)):
                p, t, _ = orc.list_schedule_alg1(s, o, M, orders[c])
                assert tel[c] == t and (starts[c] == p).all(), (o.tolist(), orders[c].tolist())
    # the stated pair on its own, checked by hand: round 37 is the first over budget, and B's ramp
    # has to drop by 196 - 195 = 1 there while A's peak (round 39: 140 + 60 = 200) asks for 5
    s, o = np.array([100, 20], dtype=np.int32), np.array([40, 60], dtype=np.int32)
    with kv.Scheduler(s, o, M) as h:
        tel, _, starts = h.eval_batch(kv.CAND_ORDER, np.array([[0, 1]], dtype=np.int32), want_starts=True)
    assert starts[0].tolist() == [0, 5] and tel[0] == 40 + 65
    assert orc.list_schedule_alg1(s, o, M, [0, 1])[0].tolist() == [0, 5]


@pytest.mark.parametrize("omax", [100, 127, 128, 129, 255, 256, 257, 511, 512, 513, 1023, 1024, 1025, 1500, 3000])
def test_orders_every_simulator_shape(omax):
    """Window lengths around each register count's limit, and the hybrid simulator beyond 1025."""
    rng = np.random.default_rng(omax)
    n, M = 90, 4 * omax
    s = rng.integers(1, omax, n).astype(np.int32)
    o = rng.integers(1, omax + 1, n).astype(np.int32)
    o[:6] = [omax, omax - 1, 1, 2, 3, omax]
    s[::11] = M - o[::11]
    orders = np.stack([rng.permutation(n) for _ in range(4)]).astype(np.int32)
    with kv.Scheduler(s, o, M) as h:
        tel, _, starts = h.eval_batch(kv.CAND_ORDER, orders, want_starts=True)
        h.set_base_order(orders[0])
        codes = all_codes(n)[::37]
        mtel, _, _ = h.eval_batch(kv.CAND_MOVE, codes)
    for c in range(4):
        p, tt, _ = orc.list_schedule_rounds(s, o, M, orders[c])
        assert tel[c] == tt and (starts[c] == p).all()
    assert (mtel == oracle_moves(s, o, M, orders[0], codes)).all()


@pytest.mark.parametrize("sim", ["smem", "hybrid"])
def test_simulators_with_shared_memory_timelines(sim, monkeypatch):
    """The all-shared-memory simulator and the hybrid one (33 registers per lane + a shared-memory ring
    for the rounds after them), each forced for every window length: short windows that never reach
    the ring, windows that end in its first chunk, windows over most of it, waits longer than the
    whole state; explicit orders with start times, moves from snapshots, and the policy sweep."""
    monkeypatch.setenv("KVSCHED_SIM", sim)
    for omax in (1, 3, 40, 300, 1025, 1026, 1057, 1100, 2500, 4096):
        rng = np.random.default_rng(1000 + omax)
        n, M = 70, 4 * omax + 8
        s = rng.integers(1, M - omax, n).astype(np.int32)
        o = rng.integers(1, omax + 1, n).astype(np.int32)
        o[:6] = [omax, max(1, omax - 1), 1, min(2, omax), min(33, omax), omax]
        s[::9] = M - o[::9]                                   # requests that need the machine alone
        orders = np.stack([rng.permutation(n) for _ in range(3)]).astype(np.int32)
        with kv.Scheduler(s, o, M) as h:
            tel, _, starts = h.eval_batch(kv.CAND_ORDER, orders, want_starts=True)
            h.set_base_order(orders[0])
            codes = all_codes(n)[::53]
            mtel, _, _ = h.eval_batch(kv.CAND_MOVE, codes)
        for c in range(3):
            p, tt, _ = orc.list_schedule_rounds(s, o, M, orders[c])
            assert tel[c] == tt and (starts[c] == p).all(), (sim, omax, c)
        assert (mtel == oracle_moves(s, o, M, orders[0], codes)).all(), (sim, omax)
    # policy sweep (one single-warp CTA per instance and policy) on the same simulator class
    rng = np.random.default_rng(77)
    B, n, M = 6, 60, 6000
    s = rng.integers(1, 3000, (B, n)).astype(np.int32)
    o = rng.integers(1, 1500, (B, n)).astype(np.int32)
    pol = np.array([kv.POLICY_FCFS, kv.POLICY_SOF, kv.POLICY_TOTAL_SIZE, kv.POLICY_SORTED_F], dtype=np.int32)
    with kv.Scheduler.batch(s, o, M) as h:
        tel, _, _ = h.eval_batch(kv.CAND_POLICY, pol)
    for b in range(B):
        refs = [orc.policy_order(s[b], o[b], orc.FCFS), orc.policy_order(s[b], o[b], orc.SHORTEST_OUTPUT_FIRST),
                orc.policy_order(s[b], o[b], orc.TOTAL_SIZE_FIRST), orc.sorted_f_prefix(s[b], o[b], M)[0]]
        for k, order in enumerate(refs):
            assert tel[b, k] == orc.list_schedule_rounds(s[b], o[b], M, order)[1], (sim, b, k)


def test_orders_mixed_1k():
    inst = W.mixed_1k()
    orders = W.random_permutations(inst.n, 6, seed=9)
    orders[0] = orc.policy_order(inst.s, inst.o, orc.SHORTEST_OUTPUT_FIRST)
    orders[1] = orc.policy_order(inst.s, inst.o, orc.TOTAL_SIZE_FIRST)
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        tel, _, starts = h.eval_batch(kv.CAND_ORDER, orders, want_starts=True)
    for c in range(len(orders)):
        p, t, _ = orc.list_schedule_rounds(inst.s, inst.o, inst.M, orders[c])
        assert tel[c] == t and (starts[c] == p).all()
    p, t, _ = orc.list_schedule_alg1(inst.s, inst.o, inst.M, orders[1])      # literal Algorithm 1 once
    assert tel[1] == t


# ------------------------------------------------------------------------------------ MOVE
def test_moves_full_neighbourhood_tiny_backlog():
    inst = W.tiny()
    base, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
    codes = all_codes(inst.n)
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        h.set_base_order(base)
        tel, _, starts = h.eval_batch(kv.CAND_MOVE, codes, want_starts=True)
    ref = oracle_moves(inst.s, inst.o, inst.M, base, codes)
    assert (tel == ref).all()
    for c in (0, 5, 119, 120, 200, len(codes) - 1):
        cand = orc.apply_move(base, *orc.decode_move(inst.n, int(codes[c])))
        assert (starts[c] == orc.list_schedule_alg1(inst.s, inst.o, inst.M, cand)[0]).all()


def test_moves_random_small_instances_all_codes():
    rng = np.random.default_rng(3)
    for trial in range(25):
        n = int(rng.integers(2, 40))
        M = int(rng.integers(10, 200))
        s, o = rand_instance(rng, n, M, M // 2, max(1, M // 3))
        base = rng.permutation(n).astype(np.int32)
        codes = all_codes(n)
        with kv.Scheduler(s, o, M) as h:
            h.set_base_order(base)
            tel, _, _ = h.eval_batch(kv.CAND_MOVE, codes)
        assert (tel == oracle_moves(s, o, M, base, codes)).all()


def test_moves_sampled_codes_mixed_1k_and_10k():
    for inst, count in ((W.mixed_1k(), 1500), (W.mixed_10k(), 160)):
        base, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
        n = inst.n
        total = n * (n - 1) // 2 + n * (n - 1)
        codes = (W.u64(77, 0, np.arange(count)) % np.uint64(total)).astype(np.int64)
        codes[:4] = [0, n * (n - 1) // 2 - 1, n * (n - 1) // 2, total - 1]
        with kv.Scheduler(inst.s, inst.o, inst.M) as h:
            h.set_base_order(base)
            tel, _, _ = h.eval_batch(kv.CAND_MOVE, codes)
        assert (tel == oracle_moves(inst.s, inst.o, inst.M, base, codes)).all()


def test_sweep_in_the_benchmarks_launch_configuration():
    """The launch the benchmark times: one sweep of 4,194,304 sampled moves of the Sorted-F order of
    the 10,000-request backlog on the handle's stream, reduced to its best (TEL, index) pair without
    a per-candidate output (TELs stay in launch-slot order inside the library).  The same sweep
    with the TELs dumped: sampled outputs against the oracle one by one; the reduced pair of both
    sweeps against an arg-min of the dumped TELs on the host; and, as a property that holds at
    any size, no candidate beats the sum of decode lengths."""
    import torch
    inst = W.mixed_10k()
    count, seed, it = 1 << 22, 20250806, 3
    dev = torch.device("cuda", 0)
    tel = torch.empty(count, dtype=torch.int64, device=dev)
    best = torch.zeros(2, dtype=torch.int64, device=dev)
    best_dump = torch.zeros(2, dtype=torch.int64, device=dev)
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        h.sorted_f_dev()
        h.sweep_dev(count, best, sampled=True, seed=seed, iteration=it, first_code=0)
        h.sweep_dev(count, best_dump, sampled=True, seed=seed, iteration=it, first_code=0, tel_out=tel)
        h.sync()
        order = h.get_base_order()
    tels = tel.cpu().numpy()
    r_order, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
    assert (order == r_order).all()
    picks = np.concatenate([[0, 1, count - 1], (W.u64(5, 1, np.arange(45)) % np.uint64(count)).astype(np.int64)])
    mv = [orc.sample_move(inst.n, seed, it, int(m)) for m in picks]
    ref = orc.eval_moves(inst.s, inst.o, inst.M, r_order, [m[0] for m in mv], [m[1] for m in mv], [m[2] for m in mv])
    assert (tels[picks] == ref).all()
    k = int(np.argmin(tels))                                   # first minimum = lowest index
    assert best_dump.cpu().tolist() == [int(tels[k]), k]
    assert best.cpu().tolist() == [int(tels[k]), k]
    assert tels.min() >= int(inst.o.sum())                     # every request completes no earlier than its own o


# ------------------------------------------------------------------------------------ Sorted-F
def test_sorted_f_matches_oracle():
    rng = np.random.default_rng(4)
    cases = [W.tiny(), W.mixed_1k(), W.mixed_10k(), W.paper_scale()]
    for trial in range(30):
        n = int(rng.integers(1, 400))
        M = int(rng.integers(10, 2000))
        s, o = rand_instance(rng, n, M, M // 2, max(1, M // 3))
        cases.append(W.Instance("rand", s, o, M))
    ties = W.Instance("ties", np.array([3, 3, 1, 5, 3, 1] * 20, dtype=np.int32), np.array([2, 2, 4, 2, 2, 4] * 20, dtype=np.int32), 37)
    cases.append(ties)
    for inst in cases:
        with kv.Scheduler(inst.s, inst.o, inst.M) as h:
            order, offs, tel = h.sorted_f()
            assert (h.get_base_order() == order).all()
        r_order, r_offs = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
        assert (offs == r_offs).all(), inst.name
        assert (order == r_order).all(), inst.name
        assert tel == orc.list_schedule_rounds(inst.s, inst.o, inst.M, r_order)[1]


def test_sorted_f_example1(golden):
    s = np.array([63] + [1] * 21, dtype=np.int32)
    o = np.array([1] + [2] * 21, dtype=np.int32)
    with kv.Scheduler(s, o, 64) as h:
        order, offs, tel = h.sorted_f()
    assert offs.tolist() == [0, 21, 22] and order[-1] == 0 and tel == golden["example1_tel_sortedf"]


def test_sorted_f_local_swap_matches_oracle():
    """Sorted-F with Algorithm 3 (Local Swap Search) as Phase-1 solver: batches, order and TEL."""
    rng = np.random.default_rng(44)
    cases = [W.tiny(), W.mixed_1k(), W.paper_scale(), W.mixed_10k()]
    for trial in range(40):
        n = int(rng.integers(1, 300))
        M = int(rng.integers(10, 1500))
        s, o = rand_instance(rng, n, M, M // 2, max(1, M // 3))
        cases.append(W.Instance("rand", s, o, M))
    cases.append(W.Instance("ties", np.array([4, 4, 6, 8] * 30, dtype=np.int32), np.array([6, 6, 4, 2] * 30, dtype=np.int32), 50))
    cases.append(W.Instance("ex1", np.array([63] + [1] * 21, dtype=np.int32), np.array([1] + [2] * 21, dtype=np.int32), 64))
    total_swaps = 0
    for inst in cases:
        with kv.Scheduler(inst.s, inst.o, inst.M) as h:
            order, offs, tel = h.sorted_f_local_swap()
            assert (h.get_base_order() == order).all()
        r_order, r_offs, swaps = orc.sorted_f_local_swap(inst.s, inst.o, inst.M)
        total_swaps += swaps
        assert (offs == r_offs).all(), inst.name
        assert (order == r_order).all(), inst.name
        assert tel == orc.list_schedule_rounds(inst.s, inst.o, inst.M, r_order)[1]
    assert total_swaps > 1000                                   # the improvement loop really ran


def test_sorted_f_exact_dp_matches_oracle():
    """Sorted-F with Algorithm 2 (exact DP) as Phase-1 solver: same batches, members and TEL as the
    oracle's DP (which is itself checked against subset enumeration)."""
    rng = np.random.default_rng(45)
    cases = [W.tiny(), W.Instance("ex1", np.array([63] + [1] * 21, dtype=np.int32), np.array([1] + [2] * 21, dtype=np.int32), 64)]
    for trial in range(25):
        n = int(rng.integers(1, 60))
        M = int(rng.integers(10, 400))
        s, o = rand_instance(rng, n, M, M // 2, max(1, M // 3))
        cases.append(W.Instance("rand", s, o, M))
    big = W.mixed_backlog(100, 77, 16492, chat_s=(2.48, 1.58, 1, 4096), chat_o=(3.76, 1.17, 1, 2048), doc_s=(500, 4800), doc_o=(30, 560))
    cases.append(big)                                           # the paper's recommended limit, n = 100
    cases.append(W.Instance("ties", np.array([4, 4, 6, 8] * 12, dtype=np.int32), np.array([6, 6, 4, 2] * 12, dtype=np.int32), 50))
    for inst in cases:
        with kv.Scheduler(inst.s, inst.o, inst.M) as h:
            order, offs, tel = h.sorted_f_dp()
        r_order, r_offs = orc.sorted_f_exact(inst.s, inst.o, inst.M, orc.DP)
        assert (offs == r_offs).all(), inst.name
        assert (order == r_order).all(), inst.name
        assert tel == orc.list_schedule_rounds(inst.s, inst.o, inst.M, r_order)[1]
    with kv.Scheduler(np.ones(200, dtype=np.int32), np.ones(200, dtype=np.int32), 10) as h:
        with pytest.raises(kv.SchedError) as e:
            h.sorted_f_dp()
        assert e.value.code == kv.E_UNSUPPORTED


def test_sorted_f_quantile_greedy_matches_oracle():
    """Sorted-F with Algorithm 4 (Quantile Greedy Selection) as Phase-1 solver: batches, order, TEL."""
    rng = np.random.default_rng(46)
    cases = [W.tiny(), W.mixed_1k(), W.paper_scale(), W.mixed_10k()]
    for trial in range(60):
        n = int(rng.integers(1, 400))
        M = int(rng.integers(10, 3000))
        s, o = rand_instance(rng, n, M, M // 2, max(1, M // 3))
        cases.append(W.Instance("rand", s, o, M))
    # more than one 1024-position tile in both first-fit walks and in the hand-out
    s, o = rand_instance(rng, 5000, 60000, 40, 30)
    cases.append(W.Instance("many_small", s, o, 60000))
    # many equal ratios and equal sizes: the stable orders decide
    cases.append(W.Instance("ties", np.array([4, 4, 6, 8, 2, 3] * 40, dtype=np.int32), np.array([4, 6, 4, 2, 2, 3] * 40, dtype=np.int32), 90))
    cases.append(W.Instance("ex1", np.array([63] + [1] * 21, dtype=np.int32), np.array([1] + [2] * 21, dtype=np.int32), 64))
    cases.append(W.Instance("one", np.array([3], dtype=np.int32), np.array([2], dtype=np.int32), 5))
    # ratios one part in 2^30 apart: r0 = k/(2k-1), r1 = (k+1)/(2k+1) with k = 2^14
    k = 1 << 14
    cases.append(W.Instance("close", np.array([k - 1, k, 9], dtype=np.int32), np.array([k, k + 1, 1], dtype=np.int32), 10 + 2 * k + 1))
    for idx, inst in enumerate(cases):
        seed = 1000 + idx
        with kv.Scheduler(inst.s, inst.o, inst.M) as h:
            order, offs, tel = h.sorted_f_quantile(seed)
            assert (h.get_base_order() == order).all()
        r_order, r_offs = orc.sorted_f_quantile(inst.s, inst.o, inst.M, seed)
        assert (offs == r_offs).all(), inst.name
        assert (order == r_order).all(), inst.name
        assert tel == orc.list_schedule_rounds(inst.s, inst.o, inst.M, r_order)[1]
    # a different seed draws different samples
    inst = W.mixed_1k()
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        a = h.sorted_f_quantile(1)[0]
        b = h.sorted_f_quantile(2)[0]
    assert (a != b).any()
    # the exact ratio key needs 2 bits(M) + bits(max o) <= 63
    with kv.Scheduler(np.array([5, 7], dtype=np.int32), np.array([512, 3], dtype=np.int32), 1 << 29) as h:
        with pytest.raises(kv.SchedError) as e:
            h.sorted_f_quantile(0)
        assert e.value.code == kv.E_UNSUPPORTED


def _online_rows(instances):
    n_max = max(len(x[0]) for x in instances)
    B = len(instances)
    a = np.zeros((B, n_max), dtype=np.int32); s = np.ones((B, n_max), dtype=np.int32); o = np.ones((B, n_max), dtype=np.int32)
    n_each = np.zeros(B, dtype=np.int32)
    for b, (ai, si, oi) in enumerate(instances):
        n = len(ai)
        n_each[b] = n
        a[b, :n], s[b, :n], o[b, :n] = ai, si, oi
    return n_each, a, s, o


ONLINE = (kv.POLICY_FCFS, kv.POLICY_SOF, kv.POLICY_SORTED_F)


def test_online_policies_match_oracle_on_small_streams():
    """Section 6.2's online policies on many small arrival streams, several refresh periods and
    look-ahead caps: every start time and every total latency."""
    rng = np.random.default_rng(61)
    M = 120
    instances = []
    for trial in range(48):
        n = int(rng.integers(1, 70))
        s, o = rand_instance(rng, n, M, M // 2, max(2, M // 4))
        spread = int(rng.choice([0, n // 2 + 1, 3 * n, 20 * n]))           # all at once ... underloaded
        a = np.sort(rng.integers(0, spread + 1, n)).astype(np.int32)
        instances.append((a, s, o))
    # the hand-worked streams of the CPU tests (M = 10 there; here they run in a launch of their own)
    n_each, a, s, o = _online_rows(instances)
    for policy in ONLINE:
        for period, lookahead in ((10, 300), (1, 1), (3, 2), (7, 5), (1 << 30, 1000)):
            starts, lat, _ = kv.online_simulate(n_each, a, s, o, M, policy, period, lookahead)
            for b, (ai, si, oi) in enumerate(instances):
                p, tot = orc.online_schedule(ai, si, oi, M, policy, period, lookahead)
                n = len(ai)
                assert (starts[b, :n] == p).all(), (policy, period, lookahead, b)
                assert (starts[b, n:] == -1).all()
                assert lat[b] == tot
            if policy != kv.POLICY_SORTED_F:
                break                                                     # the parameters only matter to Sorted-F-Online
    hand = [([0, 0, 0, 1, 2, 6], [1, 1, 6, 1, 2, 3], [2, 2, 1, 1, 1, 2]), ([0, 0, 0, 0, 1], [5, 6, 6, 7, 1], [4, 3, 2, 2, 1])]
    n_each, a, s, o = _online_rows(hand)
    starts, lat, _ = kv.online_simulate(n_each, a, s, o, 10, kv.POLICY_SORTED_F, 3, 2)
    assert starts[0].tolist() == [0, 0, 3, 2, 2, 6] and lat[0] == 13
    starts, lat, _ = kv.online_simulate(n_each, a, s, o, 10, kv.POLICY_SORTED_F, 2, 10)
    assert starts[1].tolist()[:5] == [7, 4, 0, 2, 2] and lat[1] == 26


def test_online_poisson_streams_match_oracle():
    """The paper's online experiment in small (Poisson arrivals, the three policies, period 10,
    look-ahead 300) and two full-size streams (4000 iterations, rates 0.11 and 0.30)."""
    streams = [W.online_poisson(lam, horizon=600, seed=20 + k) for k, lam in enumerate((0.05, 0.09, 0.13, 0.21, 0.30, 0.5))]
    streams += [W.online_poisson(0.11, seed=31), W.online_poisson(0.30, seed=32)]
    M = streams[0].M
    n_each, a, s, o = _online_rows([(x.a, x.s, x.o) for x in streams])
    totals = {}
    for policy in ONLINE:
        starts, lat, ms = kv.online_simulate(n_each, a, s, o, M, policy)
        for b, x in enumerate(streams):
            p, tot = orc.online_schedule(x.a, x.s, x.o, M, policy)
            assert (starts[b, :x.n] == p).all(), (policy, x.name)
            assert lat[b] == tot
        totals[policy] = lat
    # overloaded full-size stream: Sorted-F-Online < shortest decode first < FCFS (Section 7)
    assert totals[kv.POLICY_SORTED_F][-1] < totals[kv.POLICY_SOF][-1] < totals[kv.POLICY_FCFS][-1]


def test_online_argument_errors():
    n_each, a, s, o = _online_rows([([0, 1], [2, 2], [1, 1])])
    for bad in (dict(policy=kv.POLICY_TOTAL_SIZE), dict(period=0), dict(lookahead=0)):
        args = dict(policy=kv.POLICY_FCFS, period=10, lookahead=300); args.update(bad)
        with pytest.raises(kv.SchedError) as e:
            kv.online_simulate(n_each, a, s, o, 10, args["policy"], args["period"], args["lookahead"])
        assert e.value.code == kv.E_INVAL
    with pytest.raises(kv.SchedError) as e:
        kv.online_simulate(n_each, a[:, ::-1].copy(), s, o, 10, kv.POLICY_FCFS)        # arrivals decrease
    assert e.value.code == kv.E_INVAL
    with pytest.raises(kv.SchedError) as e:
        kv.online_simulate(n_each, a, s, o, 2, kv.POLICY_FCFS)                          # s + o > M
    assert e.value.code == kv.E_INVAL
    with pytest.raises(kv.SchedError) as e:
        kv.online_simulate(n_each, a, s, o, 10, kv.POLICY_SORTED_F, 10, 5000)           # look-ahead beyond the build's cap
    assert e.value.code == kv.E_UNSUPPORTED


def _amin_rows(instances):
    """instances: list of (s, lower, o, order) -> padded [B, n_max] rows."""
    n_max = max(len(x[0]) for x in instances)
    B = len(instances)
    s = np.ones((B, n_max), dtype=np.int32); lo = np.ones((B, n_max), dtype=np.int32); o = np.ones((B, n_max), dtype=np.int32)
    order = np.zeros((B, n_max), dtype=np.int32)
    n_each = np.zeros(B, dtype=np.int32)
    for b, (si, li, oi, ordi) in enumerate(instances):
        n = len(si)
        n_each[b] = n
        s[b, :n], lo[b, :n], o[b, :n], order[b, :n] = si, li, oi, ordi
    return n_each, s, lo, o, order


def test_amin_small_scenarios_match_the_set_form_oracle():
    """Algorithm 5's executor against the oracle that re-derives every projection from the sets:
    every final start time, TEL, eviction count and peak memory; tight and loose memories, exact,
    mild and crude lower bounds (l = 1 for everybody included), and the hand-worked cases."""
    rng = np.random.default_rng(71)
    for M in (60, 150):
        instances = []
        for trial in range(60):
            n = int(rng.integers(1, 60))
            s, o = rand_instance(rng, n, M, M // 2, max(2, M // int(rng.integers(2, 6))))
            kind = trial % 4
            if kind == 0: lower = o.copy()
            elif kind == 1: lower = np.ones(n, dtype=np.int32)
            else: lower = np.clip(np.floor(o * rng.uniform(0.0 if kind == 2 else 0.6, 1.0, n)), 1, o).astype(np.int32)
            instances.append((s, lower, o, rng.permutation(n).astype(np.int32)))
        n_each, s, lo, o, order = _amin_rows(instances)
        starts, tel, ev, peak, _ = kv.amin_simulate(n_each, s, lo, o, M, order)
        total_ev = 0
        for b, (si, li, oi, ordi) in enumerate(instances):
            p, rtel, rev, rpeak = orc.amin_schedule(si, li, oi, M, ordi)
            n = len(si)
            assert (starts[b, :n] == p).all(), (M, b)
            assert (starts[b, n:] == -1).all()
            assert (tel[b], ev[b], peak[b]) == (rtel, rev, rpeak), (M, b)
            if b % 4 == 0:
                assert ev[b] == 0
            total_ev += rev
        assert total_ev > 100
    hand = [([2, 3], [2, 1], [4, 2], [0, 1]), ([2, 3], [3, 1], [4, 3], [0, 1]), ([2, 3, 1], [3, 1, 1], [4, 3, 1], [0, 1, 2])]
    n_each, s, lo, o, order = _amin_rows(hand)
    starts, tel, ev, peak, _ = kv.amin_simulate(n_each, s, lo, o, 8, order)
    assert starts[0, :2].tolist() == [2, 0] and (tel[0], ev[0], peak[0]) == (8, 1, 7)
    assert starts[1, :2].tolist() == [0, 4] and (tel[1], ev[1], peak[1]) == (11, 1, 7)
    assert starts[2].tolist() == [0, 4, 4] and ev[2] == 1


def test_amin_backlogs_of_paper_size_match_the_per_round_oracle():
    """Backlogs of the size of the paper's experiments (n = 2000, M = 16,492) and of the 1,000-request
    mixture, lists from Phase 1 on the lower bounds, interval predictions of several widths
    (l = ceil(gamma o)): the whole of Sorted-F + A_min against the oracle (Phase 1 on the lower
    bounds, then the per-round executor); with exact predictions it is Sorted-F itself."""
    for inst, gammas in ((W.paper_scale(), (1.0, 0.8, 0.5)), (W.mixed_1k(), (0.9, 0.3))):
        rng = np.random.default_rng(5)
        for gamma in gammas:
            lower = np.clip(np.ceil(inst.o * rng.uniform(gamma, 1.0, inst.n)), 1, inst.o).astype(np.int32)
            for phase1 in (0, 1):
                order, starts, tel, ev, peak = kv.sorted_f_amin(inst.s, lower, inst.o, inst.M, phase1)
                if phase1 == 0:
                    r_order = orc.sorted_f_prefix(inst.s, lower, inst.M)[0]
                else:
                    r_order = orc.sorted_f_local_swap(inst.s, lower, inst.M)[0]
                assert (order == r_order).all()
                p, rtel, rev, rpeak = orc.amin_schedule_rounds(inst.s, lower, inst.o, inst.M, r_order)
                assert (starts == p).all() and (tel, ev, peak) == (rtel, rev, rpeak), (inst.name, gamma, phase1)
                assert peak <= inst.M
                if gamma == 1.0:
                    assert ev == 0 and tel == orc.list_schedule_rounds(inst.s, inst.o, inst.M, r_order)[1]
                else:
                    assert ev > 0


def test_amin_argument_errors():
    n_each, s, lo, o, order = _amin_rows([([2, 3], [1, 1], [4, 2], [0, 1])])
    with pytest.raises(kv.SchedError) as e:
        kv.amin_simulate(n_each, s, o + 1, o, 8, order)                     # lower bound above the length
    assert e.value.code == kv.E_INVAL
    with pytest.raises(kv.SchedError) as e:
        kv.amin_simulate(n_each, s, lo, o, 5, order)                        # s + o > M
    assert e.value.code == kv.E_INVAL
    with pytest.raises(kv.SchedError) as e:
        kv.amin_simulate(n_each, s, lo, o, 8, np.zeros_like(order))         # not a permutation
    assert e.value.code == kv.E_NOT_PERMUTATION
    big = np.full((1, 2), 9000, dtype=np.int32)
    with pytest.raises(kv.SchedError) as e:
        kv.amin_simulate(n_each, s, big, big, 1 << 20, order)               # decode beyond the build's cap
    assert e.value.code == kv.E_UNSUPPORTED
    with pytest.raises(kv.SchedError) as e:
        kv.sorted_f_amin([2, 3], [1, 1], [4, 2], 8, phase1=7)
    assert e.value.code == kv.E_INVAL


def test_tiny_backlog_all_solvers_and_brute_force():
    """n = 16: prefix-F, Algorithm 3 and the exact DP orders, a full swap search from the DP order,
    and all 8! orders of the first 8 requests against the oracle's brute force."""
    import itertools
    inst = W.tiny()
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        o_dp, offs_dp, tel_dp = h.sorted_f_dp()
        r_dp, r_offs = orc.sorted_f_exact(inst.s, inst.o, inst.M, orc.DP)
        assert (o_dp == r_dp).all() and (offs_dp == r_offs).all()
        final, tel, done, trace = h.local_search(kv.NBHD_SWAP, 100)       # starts from the DP order
        r_final, r_tel, r_done, r_trace = orc.local_search(inst.s, inst.o, inst.M, orc.SWAP, 100, r_dp)
        assert (final == r_final).all() and tel == r_tel and done == r_done and (trace == r_trace).all()
        assert tel <= tel_dp
    s8, o8 = inst.s[:8], inst.o[:8]
    perms = np.array(list(itertools.permutations(range(8))), dtype=np.int32)
    with kv.Scheduler(s8, o8, inst.M) as h:
        tels, _, _ = h.eval_batch(kv.CAND_ORDER, perms)
        dp8, _, tel8 = h.sorted_f_dp()
    best, best_order = orc.bruteforce_best_order(s8, o8, inst.M)
    assert tels.min() == best and (perms[int(np.argmin(tels))] == best_order).all()
    opt, _ = orc.bruteforce_opt(s8, o8, inst.M, best + 1)
    assert opt <= best <= tel8 < 48 * opt                              # Theorem 3's factor


def test_sorted_g_prefill_weight_matches_oracle():
    rng = np.random.default_rng(46)
    cases = [W.mixed_1k(), W.paper_scale()]
    for trial in range(20):
        n = int(rng.integers(1, 300))
        M = int(rng.integers(10, 1500))
        s, o = rand_instance(rng, n, M, M // 2, max(1, M // 3))
        cases.append(W.Instance("rand", s, o, M))
    for inst in cases:
        with kv.Scheduler(inst.s, inst.o, inst.M) as h:
            for a_num, a_den in ((1, 1), (13, 1000), (5, 1), (0, 3)):
                h.set_prefill_weight(a_num, a_den)
                order, offs, tel = h.sorted_f()
                r_order, r_offs = orc.sorted_g_prefix(inst.s, inst.o, inst.M, a_num, a_den)
                assert (offs == r_offs).all() and (order == r_order).all(), (inst.name, a_num, a_den)
                assert tel == orc.list_schedule_rounds(inst.s, inst.o, inst.M, r_order)[1]
                order, offs, tel = h.sorted_f_local_swap()
                r_order, r_offs = orc.sorted_g_local_swap(inst.s, inst.o, inst.M, a_num, a_den)
                assert (offs == r_offs).all() and (order == r_order).all(), (inst.name, a_num, a_den)
            with pytest.raises(kv.SchedError):
                h.set_prefill_weight(-1, 1)
            with pytest.raises(kv.SchedError):
                h.set_prefill_weight(1, 0)


# ------------------------------------------------------------------------------------ POLICY
def test_policy_sweep_small_batch():
    s, o, M = W.policy_sweep(num_instances=24, n_each=256)
    pols = np.array([kv.POLICY_SORTED_F, kv.POLICY_FCFS, kv.POLICY_SOF, kv.POLICY_TOTAL_SIZE], dtype=np.int32)
    with kv.Scheduler.batch(s, o, M) as h:
        tel, feas, starts = h.eval_batch(kv.CAND_POLICY, pols, want_feasible=True, want_starts=True)
    assert tel.shape == (24, 4) and feas.all()
    for b in range(24):
        refs = [orc.sorted_f_prefix(s[b], o[b], M)[0], orc.policy_order(s[b], o[b], orc.FCFS),
                orc.policy_order(s[b], o[b], orc.SHORTEST_OUTPUT_FIRST), orc.policy_order(s[b], o[b], orc.TOTAL_SIZE_FIRST)]
        for k, order in enumerate(refs):
            p, t, _ = orc.list_schedule_rounds(s[b], o[b], M, order)
            assert tel[b, k] == t
            assert (starts[b, k] == p).all()


def test_policy_on_single_instance_handle_and_odd_sizes():
    rng = np.random.default_rng(6)
    for n in (1, 2, 31, 33, 100):
        M = 300
        s, o = rand_instance(rng, n, M, 100, 60)
        with kv.Scheduler(s, o, M) as h:
            tel, _, _ = h.eval_batch(kv.CAND_POLICY, np.array([3, 2, 1, 0], dtype=np.int32))
        refs = [orc.sorted_f_prefix(s, o, M)[0], orc.policy_order(s, o, 2), orc.policy_order(s, o, 1), orc.policy_order(s, o, 0)]
        assert tel[0].tolist() == [orc.list_schedule_alg1(s, o, M, r)[1] for r in refs]


# ------------------------------------------------------------------------------------ START_TIMES
def test_start_times_checker():
    rng = np.random.default_rng(7)
    for trial in range(20):
        n = int(rng.integers(1, 50))
        M = int(rng.integers(20, 200))
        s, o = rand_instance(rng, n, M, M // 2, max(1, M // 4))
        good = orc.list_schedule_alg1(s, o, M, rng.permutation(n))[0]
        cands = [good]
        for _ in range(6):                                 # perturbed starts: some overflow, some do not
            p = good.copy()
            k = rng.integers(0, n, max(1, n // 4))
            p[k] = np.maximum(0, p[k] + rng.integers(-5, 6, len(k)))
            cands.append(p)
        cands.append(np.zeros(n, dtype=np.int64))          # everything at once
        cands.append(good + 1000)                          # far beyond the ring length
        cands = np.stack(cands).astype(np.int32)
        with kv.Scheduler(s, o, M) as h:
            tel, feas, _ = h.eval_batch(kv.CAND_START_TIMES, cands, want_feasible=True)
        for c in range(len(cands)):
            r = orc.check_schedule(s, o, M, cands[c])
            assert tel[c] == r["tel"] and bool(feas[c]) == r["feasible"]
        assert feas[0] == 1


# ------------------------------------------------------------------------------------ local search
def test_local_search_tiny_backlog_full_swap_sweeps():
    inst = W.tiny()
    base, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
    for nb, onb in ((kv.NBHD_SWAP, orc.SWAP), (kv.NBHD_SWAP_INSERT, orc.SWAP_INSERT)):
        with kv.Scheduler(inst.s, inst.o, inst.M) as h:
            final, tel, done, trace = h.local_search(nb, 200, order=base)
        r_final, r_tel, r_done, r_trace = orc.local_search(inst.s, inst.o, inst.M, onb, 200, base)
        assert (final == r_final).all() and tel == r_tel and done == r_done
        assert (trace == r_trace).all()


def test_local_search_random_instances_to_local_optimum():
    rng = np.random.default_rng(8)
    for trial in range(6):
        n = int(rng.integers(5, 30))
        M = int(rng.integers(30, 150))
        s, o = rand_instance(rng, n, M, M // 2, M // 4)
        start = rng.permutation(n).astype(np.int32)
        with kv.Scheduler(s, o, M) as h:
            final, tel, done, trace = h.local_search(kv.NBHD_SWAP_INSERT, 500, order=start)
        r_final, r_tel, r_done, r_trace = orc.local_search(s, o, M, orc.SWAP_INSERT, 500, start)
        assert (final == r_final).all() and tel == r_tel and done == r_done and (trace == r_trace).all()


def test_local_search_sampled_and_resume():
    inst = W.mixed_backlog(400, 21, 30000)
    base, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
    r_final, r_tel, r_done, r_trace = orc.local_search(inst.s, inst.o, inst.M, orc.SAMPLED, 4, base, seed=99, samples=300)
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        h.sorted_f()
        final, tel, done, trace = h.local_search(kv.NBHD_SAMPLED, 4, seed=99, samples_per_iter=300)
        assert (final == r_final).all() and tel == r_tel and done == r_done == 4 and (trace == r_trace).all()
        assert (h.get_base_order() == r_final).all()       # the handle keeps the result: a run can be resumed


def test_local_search_first_sweeps_mixed_1k():
    inst = W.mixed_1k()
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        base, _, tel0 = h.sorted_f()
        final, tel, done, trace = h.local_search(kv.NBHD_SWAP, 2)
    assert done == 2 and tel <= tel0
    # the accepted moves really have the TELs claimed, and the final order is what they produce
    cur = base
    for code, best in trace:
        cand = orc.apply_move(cur, *orc.decode_move(inst.n, int(code)))
        assert orc.list_schedule_rounds(inst.s, inst.o, inst.M, cand)[1] == best
        if best < orc.list_schedule_rounds(inst.s, inst.o, inst.M, cur)[1]:
            cur = cand
    assert (final == cur).all()
    # no sampled neighbour of the first sweep beats the reported best
    n = inst.n
    codes = (W.u64(5, 0, np.arange(400)) % np.uint64(n * (n - 1) // 2)).astype(np.int64)
    assert oracle_moves(inst.s, inst.o, inst.M, base, codes).min() >= trace[0][1]


def test_sharded_search_driver_on_one_gpu_equals_the_library_search():
    """parallel.sharded_local_search with one rank (sweep + sched_accept_move per iteration) against
    sched_local_search and the oracle; then the same search with the sweep cut into three shares that
    are reduced on the host, which is what several ranks do."""
    from paper_2508_06133_b200 import parallel as par
    rng = np.random.default_rng(91)
    n, M = 40, 300
    s, o = rand_instance(rng, n, M, 120, 60)
    start = rng.permutation(n).astype(np.int32)
    for nbhd, iters, samples in ((kv.NBHD_SWAP_INSERT, 60, 0), (kv.NBHD_SAMPLED, 12, 200)):
        r_order, r_tel, r_done, r_trace = orc.local_search(s, o, M, nbhd, iters, start, seed=3, samples=samples)
        with kv.Scheduler(s, o, M) as h:
            h.set_base_order(start)
            tel, done, trace = par.sharded_local_search(par.GpuEvaluator(h), nbhd, iters, seed=3, samples_per_iter=samples)
            assert (tel, done) == (r_tel, r_done) and (trace == r_trace).all()
            assert (h.get_base_order() == r_order).all()
        with kv.Scheduler(s, o, M) as h:                       # three shares, reduced as the ranks would
            h.set_base_order(start)
            ev = par.GpuEvaluator(h)
            total = par.neighbourhood_size(n, nbhd, samples)
            for it in range(r_done):
                pairs = [ev.sweep(*par.shard(total, r, 3), nbhd == kv.NBHD_SAMPLED, 3, it) for r in range(3)]
                best = min(pairs)                              # smallest TEL, then lowest index
                assert (best[1], best[0]) == tuple(r_trace[it])
                ev.accept(best[0], best[1], nbhd == kv.NBHD_SAMPLED, 3, it)
            assert (h.get_base_order() == r_order).all()
    # the exchange itself over NCCL (one rank: the same calls every rank of a larger job makes)
    import os
    import torch
    import torch.distributed as dist
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % (29600 + os.getpid() % 300), rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    try:
        r_order, r_tel, r_done, r_trace = orc.local_search(s, o, M, kv.NBHD_SAMPLED, 6, start, seed=8, samples=150)
        with kv.Scheduler(s, o, M) as h:
            h.set_base_order(start)
            tel, done, trace = par.sharded_local_search(par.GpuEvaluator(h), kv.NBHD_SAMPLED, 6, seed=8, samples_per_iter=150,
                                                        comm=par.TorchComm(device=torch.device("cuda", 0)))
            assert (tel, done) == (r_tel, r_done) and (trace == r_trace).all() and (h.get_base_order() == r_order).all()
    finally:
        dist.destroy_process_group()
    with kv.Scheduler(s, o, M) as h:
        h.set_base_order(start)
        base = orc.list_schedule_rounds(s, o, M, start)[1]
        assert h.accept_move(base, 0) == (False, base)         # not strictly better: refused
        with pytest.raises(kv.SchedError) as e:
            h.accept_move(base - 1, 0)                         # a TEL that move 0 does not have
        assert e.value.code == kv.E_INTERNAL
        with pytest.raises(kv.SchedError) as e:
            h.accept_move(1, n * (n - 1) // 2 + n * (n - 1))   # index outside the neighbourhood
        assert e.value.code == kv.E_INVAL


def test_cached_device_memory_is_reused_and_released():
    """Handles created and destroyed in a row take their large blocks from the library's cache (stale
    contents must not matter: every result is again the oracle's), and
    sched_release_cached_memory gives the blocks back to the driver."""
    import torch
    inst = W.mixed_1k()
    n = inst.n
    total = n * (n - 1) // 2 + n * (n - 1)
    r_order, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
    seen = []
    for rep in range(3):
        codes = (W.u64(300 + rep, 0, np.arange(500)) % np.uint64(total)).astype(np.int64)
        with kv.Scheduler(inst.s, inst.o, inst.M) as h:
            order, offs, tel = h.sorted_f()
            tels, _, _ = h.eval_batch(kv.CAND_MOVE, codes)
        assert (order == r_order).all()
        assert (tels == oracle_moves(inst.s, inst.o, inst.M, r_order, codes)).all()
        seen.append(tel)
    assert len(set(seen)) == 1
    torch.cuda.synchronize()
    free_cached = torch.cuda.mem_get_info()[0]
    kv.release_cached_memory()
    free_released = torch.cuda.mem_get_info()[0]
    assert free_released >= free_cached + (4 << 20)          # the 1,000-request snapshots alone are 4 MB
    kv.release_cached_memory()                               # nothing left: still fine
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        assert h.sorted_f()[2] == seen[0]


def test_device_pointer_candidates_are_bounds_checked_on_the_device():
    import torch
    dev = torch.device("cuda", torch.cuda.current_device())
    s, o = np.array([2, 3, 4, 5], dtype=np.int32), np.array([1, 2, 3, 1], dtype=np.int32)
    big = np.iinfo(np.int64).max
    with kv.Scheduler(s, o, 20) as h:
        # 6 swaps + 12 inserts: 0..17 valid; -1 sits next to code 0, and 18 + 2^33 * (n - 1) would wrap
        # to row 0 of the inserts if the row were narrowed to 32 bits before the range check
        codes = torch.tensor([0, 17, 18, 10 ** 12, -5, -1, 18 + (1 << 33) * 3], dtype=torch.int64, device=dev)
        tel = torch.zeros(7, dtype=torch.int64, device=dev)
        h.eval_batch_dev(kv.CAND_MOVE, 7, codes, tel)
        h.sync()
        got = tel.cpu().numpy()
        assert got[0] == oracle_moves(s, o, 20, np.arange(4), [0])[0] and got[1] == oracle_moves(s, o, 20, np.arange(4), [17])[0]
        assert (got[2:] == big).all()
        orders = torch.tensor([[3, 2, 1, 0], [0, 1, 2, 4], [0, -1, 2, 3]], dtype=torch.int32, device=dev)
        tel = torch.zeros(3, dtype=torch.int64, device=dev)
        h.eval_batch_dev(kv.CAND_ORDER, 3, orders, tel)
        h.sync()
        got = tel.cpu().numpy()
        assert got[0] == orc.list_schedule_alg1(s, o, 20, [3, 2, 1, 0])[1] and (got[1:] == big).all()
        starts = torch.tensor([[0, 0, 0, 0], [0, -3, 0, 0]], dtype=torch.int32, device=dev)
        tel = torch.zeros(2, dtype=torch.int64, device=dev)
        feas = torch.zeros(2, dtype=torch.uint8, device=dev)
        h.eval_batch_dev(kv.CAND_START_TIMES, 2, starts, tel, feas)
        h.sync()
        assert feas.cpu().numpy().tolist() == [int(orc.check_schedule(s, o, 20, [0, 0, 0, 0])["feasible"]), 0]


def test_sweep_accepts_any_8_byte_aligned_tel_array():
    """tel_out of a sweep may be a slice that starts on an odd element (8-byte but not 16-byte
    aligned); a pointer that is not 8-byte aligned is refused on the host before any launch."""
    import ctypes as C
    import torch
    dev = torch.device("cuda", torch.cuda.current_device())
    inst = W.mixed_backlog(200, 21, 20000, name="offset")
    n = inst.n
    total = n * (n - 1) // 2 + n * (n - 1)
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        h.sorted_f_dev()
        ref_tel = torch.empty(total, dtype=torch.int64, device=dev)
        ref_best = torch.zeros(2, dtype=torch.int64, device=dev)
        h.sweep_dev(total, ref_best, tel_out=ref_tel)
        for count in (total, total - 1, 1, 2):
            buf = torch.full((total + 3,), -7, dtype=torch.int64, device=dev)
            best = torch.zeros(2, dtype=torch.int64, device=dev)
            h.sweep_dev(count, best, tel_out=buf[1:1 + count])
            h.sync()
            got = buf.cpu().numpy()
            want = ref_tel[:count].cpu().numpy()
            assert (got[1:1 + count] == want).all() and got[0] == -7 and (got[1 + count:] == -7).all()
            k = int(np.argmin(want))
            assert best.cpu().tolist() == [int(want[k]), k]
        lib = kv.load()
        buf = torch.zeros(16, dtype=torch.int64, device=dev)
        best = torch.zeros(2, dtype=torch.int64, device=dev)
        launches = h.stats()[0]
        rc = lib.sched_sweep_dev(h._h, 0, 0, 0, 0, 4, C.c_void_p(buf.data_ptr() + 4), C.c_void_p(best.data_ptr()))
        assert rc == kv.E_INVAL and h.stats()[0] == launches


# ------------------------------------------------------------------------------------ errors on a live handle
def test_error_paths_on_a_handle():
    s, o = np.array([2, 3, 4], dtype=np.int32), np.array([1, 2, 3], dtype=np.int32)
    with kv.Scheduler(s, o, 20) as h:
        with pytest.raises(kv.SchedError) as e:
            h.eval_batch(kv.CAND_ORDER, np.array([[0, 1, 1]], dtype=np.int32))
        assert e.value.code == kv.E_NOT_PERMUTATION
        with pytest.raises(kv.SchedError) as e:
            h.set_base_order(np.array([0, 1, 3], dtype=np.int32))
        assert e.value.code == kv.E_NOT_PERMUTATION
        with pytest.raises(kv.SchedError) as e:
            h.eval_batch(kv.CAND_MOVE, np.array([9], dtype=np.int64))       # 3 swaps + 6 inserts = codes 0..8
        assert e.value.code == kv.E_INVAL
        with pytest.raises(kv.SchedError) as e:
            h.eval_batch(kv.CAND_POLICY, np.array([7], dtype=np.int32))
        assert e.value.code == kv.E_INVAL
        with pytest.raises(kv.SchedError) as e:
            h.eval_batch(kv.CAND_START_TIMES, np.array([[0, -1, 0]], dtype=np.int32))
        assert e.value.code == kv.E_INVAL
        with pytest.raises(kv.SchedError) as e:
            h.eval_batch(17, np.array([0], dtype=np.int32))
        assert e.value.code == kv.E_INVAL
        tel, _, _ = h.eval_batch(kv.CAND_ORDER, np.array([[2, 1, 0]], dtype=np.int32))   # still usable
        assert tel[0] == orc.list_schedule_alg1(s, o, 20, [2, 1, 0])[1]
        launches, evals = h.stats()
        assert launches > 0 and evals >= 1


def test_a_loop_cap_that_runs_out_is_reported_and_leaves_the_handle_usable():
    """With the device loops' caps lowered to zero iterations, the first request that has to wait makes
    the simulator give up: the kernel ends normally, the call returns SCHED_E_INTERNAL, nothing
    faults, and with the caps restored the same handle evaluates the same candidates correctly."""
    inst = W.mixed_backlog(400, 31, 20000, name="cap")
    orders = np.stack([np.arange(inst.n), np.arange(inst.n)[::-1]]).astype(np.int32)
    ref = [orc.list_schedule_rounds(inst.s, inst.o, inst.M, r)[1] for r in orders]
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        assert h.eval_batch(kv.CAND_ORDER, orders)[0].tolist() == ref
        kv.debug_set_loop_cap(0)
        try:
            with pytest.raises(kv.SchedError) as e:
                h.eval_batch(kv.CAND_ORDER, orders)
            assert e.value.code == kv.E_INTERNAL
            with pytest.raises(kv.SchedError) as e:
                h.sorted_f()
            assert e.value.code == kv.E_INTERNAL
        finally:
            kv.debug_set_loop_cap(-1)
        assert h.eval_batch(kv.CAND_ORDER, orders)[0].tolist() == ref
        order, _, tel = h.sorted_f()
        r_order, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
        assert (order == r_order).all() and tel == orc.list_schedule_rounds(inst.s, inst.o, inst.M, r_order)[1]
    # the hybrid and the all-shared-memory simulators, and the policy kernel, report the same way
    s2, o2, M2 = W.policy_sweep(num_instances=8)
    pols = np.array([kv.POLICY_SORTED_F, kv.POLICY_FCFS], dtype=np.int32)
    with kv.Scheduler.batch(s2, o2, M2) as h:
        good = h.eval_batch(kv.CAND_POLICY, pols)[0]
        kv.debug_set_loop_cap(0)
        try:
            with pytest.raises(kv.SchedError) as e:
                h.eval_batch(kv.CAND_POLICY, pols)
            assert e.value.code == kv.E_INTERNAL
        finally:
            kv.debug_set_loop_cap(-1)
        assert (h.eval_batch(kv.CAND_POLICY, pols)[0] == good).all()


def test_probe_peaks_are_plausible():
    """The roofline denominators come from the library's own probe kernels: every rate must be positive
    and finite, no pipe can beat the issue limit of 128 lanes per clock and SM at the top clock, the
    integer ALU pipe alone must not beat compiler-scheduled adds, and repeated calls agree."""
    import torch
    prop = torch.cuda.get_device_properties(torch.cuda.current_device())
    a = kv.probe_peaks(repeats=3)
    b = kv.probe_peaks(repeats=3)
    assert set(a) == set(kv.PROBE_NAMES)
    limit = prop.multi_processor_count * 128 * 2.2e9                 # lanes x a clock no B200 reaches
    for name in ("int_add", "int_add_max", "int_mad", "sim_mix", "int_alu"):
        assert 0 < a[name] < limit and abs(a[name] - b[name]) < 0.1 * a[name], (name, a[name], b[name])
    assert a["int_alu"] <= 1.05 * a["int_add"] and a["int_mad"] <= 1.05 * a["int_add"]
    for name in ("smem_load", "smem_store"):
        assert 0 < a[name] < prop.multi_processor_count * 256 * 2.2e9
    lib = kv.load()
    assert lib.sched_probe_peaks(None, 7, 3, None) == kv.E_INVAL
    out = np.zeros(3)
    assert lib.sched_probe_peaks(out.ctypes.data, 3, 3, None) == kv.E_INVAL


# ------------------------------------------------------------------------------------ full-size configurations
def test_policy_sweep_full_size_sampled_instances():
    """4,096 instances x 4 policies in one launch; a sample of instances is re-evaluated by the oracle."""
    s, o, M = W.policy_sweep()
    pols = np.array([kv.POLICY_SORTED_F, kv.POLICY_FCFS, kv.POLICY_SOF, kv.POLICY_TOTAL_SIZE], dtype=np.int32)
    with kv.Scheduler.batch(s, o, M) as h:
        tel, _, _ = h.eval_batch(kv.CAND_POLICY, pols)
    assert tel.shape == (4096, 4)
    for b in list(range(0, 4096, 97)) + [4095]:
        refs = [orc.sorted_f_prefix(s[b], o[b], M)[0], orc.policy_order(s[b], o[b], orc.FCFS),
                orc.policy_order(s[b], o[b], orc.SHORTEST_OUTPUT_FIRST), orc.policy_order(s[b], o[b], orc.TOTAL_SIZE_FIRST)]
        assert tel[b].tolist() == [orc.list_schedule_rounds(s[b], o[b], M, r)[1] for r in refs]
    # Sorted-F is not worse than FCFS on the bulk of these mixed backlogs
    assert (tel[:, 0] <= tel[:, 1]).mean() > 0.9


def test_mixed_1k_swap_search_to_local_optimum():
    """Sorted-F then 2-swap local search until no swap improves (n = 1,000: 499,500 neighbours per
    sweep).  Every accepted move is replayed through the oracle; the end point is checked to be a
    local optimum on a sample of its neighbourhood."""
    inst = W.mixed_1k()
    n = inst.n
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        base, _, tel0 = h.sorted_f()
        final, tel, done, trace = h.local_search(kv.NBHD_SWAP, 5000)
        assert done < 5000 and len(trace) == done
        cur, cur_tel = base, tel0
        for code, best in trace[:-1]:                              # all but the last sweep were accepted
            cur = orc.apply_move(cur, *orc.decode_move(n, int(code)))
            assert best < cur_tel
            cur_tel = int(best)
        assert trace[-1][1] >= cur_tel                             # the last sweep found nothing better
        assert (final == cur).all() and tel == cur_tel
        assert orc.list_schedule_rounds(inst.s, inst.o, inst.M, final)[1] == tel
        # spot checks of accepted TELs by the oracle, spread over the run
        cur = base
        for k, (code, best) in enumerate(trace[:-1]):
            cur = orc.apply_move(cur, *orc.decode_move(n, int(code)))
            if k % 16 == 0:
                assert orc.list_schedule_rounds(inst.s, inst.o, inst.M, cur)[1] == best
        codes = (W.u64(8, 0, np.arange(600)) % np.uint64(n * (n - 1) // 2)).astype(np.int64)
        assert oracle_moves(inst.s, inst.o, inst.M, final, codes).min() >= tel
    assert tel < tel0


def test_heavy_100k_backlog():
    """n = 100,000, o up to 4,096 (hybrid simulator, strided snapshots), int64 TELs."""
    inst = W.heavy_100k()
    n = inst.n
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        order, offs, tel = h.sorted_f()
        r_order, r_offs = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
        assert (offs == r_offs).all() and (order == r_order).all()
        p, r_tel, _ = orc.list_schedule_rounds(inst.s, inst.o, inst.M, r_order)
        assert tel == r_tel
        fcfs, _, _ = h.eval_batch(kv.CAND_ORDER, np.arange(n, dtype=np.int32)[None, :])
        assert fcfs[0] == orc.list_schedule_rounds(inst.s, inst.o, inst.M, np.arange(n))[1]
        assert fcfs[0] > 2 ** 32                                    # beyond 32 bits: TELs are int64
        total = n * (n - 1) // 2 + n * (n - 1)
        codes = (W.u64(41, 0, np.arange(6)) % np.uint64(total)).astype(np.int64)
        codes[0], codes[1] = n * (n - 1) // 2 - 1, total - 1
        mtel, _, _ = h.eval_batch(kv.CAND_MOVE, codes)
        assert (mtel == oracle_moves(inst.s, inst.o, inst.M, r_order, codes)).all()
        final, ftel, done, trace = h.local_search(kv.NBHD_SAMPLED, 2, seed=17, samples_per_iter=1 << 13)
    assert done == 2 and ftel <= tel
    cur, cur_tel = r_order, r_tel
    for it, (m, best) in enumerate(trace):
        cand = orc.apply_move(cur, *orc.sample_move(n, 17, it, int(m)))
        assert orc.list_schedule_rounds(inst.s, inst.o, inst.M, cand)[1] == best
        for mm in (0, 1, (1 << 13) - 1):                           # no sampled move beats the reported best
            c2 = orc.apply_move(cur, *orc.sample_move(n, 17, it, mm))
            assert orc.list_schedule_rounds(inst.s, inst.o, inst.M, c2)[1] >= best
        if best < cur_tel:
            cur, cur_tel = cand, best
    assert (final == cur).all() and ftel == cur_tel
