"""Do the pins bite?  Each case plants one plausible mistake in a copy of the CPU oracle (never in
the GPU code), loads the mutated library in place of the real one and checks that a named pin test
fails.  A pin that still passed would mean that part of the oracle is effectively unpinned."""
import ctypes as C
import os
import subprocess
import sys

import pytest

import oracle as orc
from tests import test_oracle_pins as pins

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(os.path.dirname(HERE), "oracle", "oracle.cpp")

MUTATIONS = [
    # (what, text in oracle.cpp, replacement, pin that must fail, needs the golden fixture)
    ("start-time convention of Algorithm 1", "p[i] = t - 1;", "p[i] = t;", "test_example1_tel", True),
    ("capacity off by one in the round-form executor", "if (U[k + j] + s[i] + j > M) { fits = false; break; }",
     "if (U[k + j] + s[i] + j >= M) { fits = false; break; }", "test_example1_tel", True),
    ("ramp term dropped in the checker", "U[p[i] + j] += (i64)s[i] + j;\n    i64 pk", "U[p[i] + j] += (i64)s[i];\n    i64 pk",
     "test_example1_checker_by_hand", True),
    ("completion time without the decode length", "for (int i = 0; i < n; ++i) total += p[i] + o[i];\n    if (tel) *tel = total;\n    if (peak)",
     "for (int i = 0; i < n; ++i) total += p[i];\n    if (tel) *tel = total;\n    if (peak)", "test_example1_checker_by_hand", True),
    ("F ties to the smaller batch", "if (kA != kB) return kA > kB ? -1 : 1;", "if (kA != kB) return kA < kB ? -1 : 1;",
     "test_example1_f_metric", True),
    ("F compared with k instead of k^2", "u128 l = (u128)sumA * (u128)kB * (u128)kB, r = (u128)sumB * (u128)kA * (u128)kA;",
     "u128 l = (u128)sumA * (u128)kB, r = (u128)sumB * (u128)kA;", "test_phase1_dp_matches_enumeration_and_lemma1", False),
    ("prefix-F memory test off by one", "mem += s[r] + o[r];\n            if (mem > M) break;\n            so += o[r];",
     "mem += s[r] + o[r];\n            if (mem >= M) break;\n            so += o[r];", "test_prefix_f_by_hand", False),
    ("insert code maps to the wrong target", "*type = 1; *i_out = i; *j_out = r < i ? r : r + 1;",
     "*type = 1; *i_out = i; *j_out = r <= i ? r : r + 1;", "test_move_codes_enumerate_the_neighbourhood", False),
    ("Algorithm 3 memory test off by one", "if (mem - size_of(X[k]) + size_of(I[p]) > M) return false;",
     "if (mem - size_of(X[k]) + size_of(I[p]) >= M) return false;", "test_local_swap_worked_by_hand", False),
    ("G-metric without the prefill term", "sw += a_num * s[r] + a_den * o[r];", "sw += a_den * o[r];",
     "test_sorted_g_reduces_to_f_and_differs_by_hand", False),
    ("Algorithm 4 quantile position", "const int q = (int)((3ll * (sample_size - 1)) / 10);", "const int q = (int)((3ll * sample_size) / 10);",
     "test_quantile_greedy_properties", False),
    ("Algorithm 4 pass 2 stops at the first misfit", "for (int r : remaining) {\n        i64 T = (i64)s[r] + o[r];\n        if (mem + T <= M) { X.push_back(r); mem += T; }\n    }",
     "for (int r : remaining) {\n        i64 T = (i64)s[r] + o[r];\n        if (mem + T <= M) { X.push_back(r); mem += T; } else break;\n    }",
     "test_quantile_greedy_worked_by_hand", False),
    ("Algorithm 4 ratio compared in floating point", "__int128 l = (__int128)o[a] * ((i64)s[b] + o[b]), r = (__int128)o[b] * ((i64)s[a] + o[a]);",
     "double l = (double)o[a] / ((double)s[a] + o[a]), r = (double)o[b] / ((double)s[b] + o[b]);", "test_quantile_greedy_worked_by_hand", False),
    ("Algorithm 4 without the output-length threshold", "if (T <= Qp && o[r] <= Qo && mem + T <= M)", "if (T <= Qp && mem + T <= M)",
     "test_quantile_greedy_worked_by_hand", False),
    ("Algorithm 4 sample of the wrong size", "int size = m / 2 > 1 ? m / 2 : 1;", "int size = (m + 1) / 2;", "test_quantile_greedy_properties", False),
    ("online: early refresh at 100 % instead of 50 %", "|| 2 * new_since >= backlog_last) {", "|| new_since >= backlog_last) {",
     "test_sorted_f_online_worked_by_hand", False),
    ("online: a refused head is skipped", "if (!fits) break;\n            for (int j = 1; j <= o[r]; ++j) U[t - 1 + j] += (i64)s[r] + j;",
     "if (!fits) continue;\n            for (int j = 1; j <= o[r]; ++j) U[t - 1 + j] += (i64)s[r] + j;", "test_online_fcfs_and_shortest_first_worked_by_hand", False),
    ("online: arrivals seen one iteration early", "if (!seen[i] && a[i] <= t - 1)", "if (!seen[i] && a[i] <= t)",
     "test_online_underloaded_requests_start_on_arrival", False),
    ("online: no look-ahead cap", "const int wn = m < lookahead ? m : lookahead;", "const int wn = m;", "test_sorted_f_online_worked_by_hand", False),
    ("online: periodic refresh never fires", "if (!computed || t - t_last >= period || was_empty", "if (!computed || was_empty",
     "test_sorted_f_online_worked_by_hand", False),
    ("A_min evicts the largest estimate", "if (state[j] == 1 && (victim < 0 || est[j] < est[victim])) victim = j;",
     "if (state[j] == 1 && (victim < 0 || est[j] > est[victim])) victim = j;", "test_amin_worked_by_hand", False),
    ("A_min estimates never grow", "else est[j] = std::max(est[j], t - p[j]);", "else est[j] = est[j];",
     "test_amin_never_exceeds_memory_and_finishes_everything", False),
    ("A_min admission off by one", "if (projected_peak(t, r, t - 1) > M) break;", "if (projected_peak(t, r, t - 1) >= M) break;",
     "test_amin_with_exact_predictions_is_algorithm_1", False),
    ("per-round A_min leaves an evicted ramp behind", "for (i64 tau = t; tau <= p[victim] + est[victim]; ++tau) proj[tau % H] -= s[victim] + tau - p[victim];",
     "for (i64 tau = t + 1; tau <= p[victim] + est[victim]; ++tau) proj[tau % H] -= s[victim] + tau - p[victim];",
     "test_amin_per_round_form_equals_the_set_form", False),
    ("per-round A_min grows an estimate without its memory", "else if (t - p[j] > est[j]) { est[j] = t - p[j]; proj[t % H] += s[j] + t - p[j]; }",
     "else if (t - p[j] > est[j]) { est[j] = t - p[j]; proj[t % H] += t - p[j]; }",
     "test_amin_per_round_form_equals_the_set_form", False),
    ("Algorithm 1's batch constraint replaced by the sum test", "if (reading == 1) feas = mem <= M;", "if (reading == 1 || reading == 0) feas = mem <= M;",
     "test_phase1_algorithm1_constraint_by_hand", False),
    ("Algorithm 1's batch constraint counts requests that have already finished", "if ((mask >> b & 1) && o[ids[b]] >= o[ids[a]]) tot += (i64)s[ids[b]] + o[ids[a]];",
     "if (mask >> b & 1) tot += (i64)s[ids[b]] + o[ids[a]];", "test_phase1_algorithm1_constraint_by_hand", False),
    ("shortest-output-first sorts by size", "std::stable_sort(order, order + n, [&](int a, int b) { return o[a] < o[b]; });",
     "std::stable_sort(order, order + n, [&](int a, int b) { return s[a] + o[a] < s[b] + o[b]; });", "test_policies", False),
]


@pytest.fixture(scope="module")
def source():
    return open(SRC).read()


_CHILD = r"""
import ctypes as C, sys
sys.path.insert(0, sys.argv[1])
import oracle as orc
from tests import test_oracle_pins as pins
from tests.conftest import load_golden
lib = C.CDLL(sys.argv[2])
lib.orc_bruteforce_opt.restype = C.c_longlong
lib.orc_bruteforce_best_order.restype = C.c_longlong
orc.lib()                      # the real library first, so that nothing rebuilds it later
orc._lib = lib
pin, needs_golden = sys.argv[3], sys.argv[4] == "1"
gold = load_golden() if needs_golden else None
fn = getattr(pins, pin)
try:
    if pin == "test_example1_tel":
        for ex in (orc.list_schedule_alg1, orc.list_schedule_rounds):
            fn(gold, ex)
    elif needs_golden:
        fn(gold)
    else:
        fn()
except (AssertionError, ValueError):
    sys.exit(0)                # the pin caught the planted mistake
sys.exit(3)                    # the pin still passes
"""


@pytest.mark.parametrize("what,old,new,pin,needs_golden", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_pin_catches_planted_mistake(tmp_path, source, what, old, new, pin, needs_golden):
    """The mutated copy runs in a child process: a planted mistake may write out of bounds, and a
    fault there must not take the test session down.  Exit code 0 = the pin failed as it should;
    a child killed by a signal (the mutated code faulted) cannot have passed the pin either."""
    assert source.count(old) == 1, "mutation site must be unique: " + what
    mutated = tmp_path / "oracle_mut.cpp"
    mutated.write_text(source.replace(old, new))
    so = tmp_path / "liboracle_mut.so"
    subprocess.check_call(["g++", "-O1", "-std=c++17", "-pthread", "-shared", "-fPIC", "-o", str(so), str(mutated)])
    root = os.path.dirname(HERE)
    r = subprocess.run([sys.executable, "-c", _CHILD, root, str(so), pin, "1" if needs_golden else "0"],
                       capture_output=True, text=True, timeout=600)
    assert r.returncode != 3, "the pin %s still passes with: %s" % (pin, what)
    assert r.returncode == 0 or r.returncode < 0, "child failed unexpectedly (%d): %s" % (r.returncode, r.stderr[-2000:])
