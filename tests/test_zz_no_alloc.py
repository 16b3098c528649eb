"""GPU check of ``sched_argmin_static_dev``, the arg-min entry point that allocates nothing.

Some users of this library cannot call the device allocator: their process has given all GPU memory
to a pool, or they run inside buffers handed to them, or they cannot afford the synchronisation an
allocation implies.  For them the reduction's scratch is a fixed array inside the library instead of
memory owned by a handle.  The result has to be identical to what the handle-based sweep reports as
its best (TEL, index) pair, also on a second call that finds the first call's leftovers in the array.
This file is collected last on purpose, so a failure here cannot hide the other tests' outcome.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_static_argmin_matches_sweep_twice_in_a_row():
    import torch
    from paper_2508_06133_b200 import binding as kv
    from paper_2508_06133_b200 import workloads as W

    dev = torch.device("cuda", torch.cuda.current_device())
    inst = W.mixed_backlog(500, 31, 40000)
    with kv.Scheduler(inst.s, inst.o, inst.M) as h:
        h.sorted_f()
        for call, (count, first) in enumerate(((70001, 0), (333, 1234))):      # many blocks, then one
            tel = torch.empty(count, dtype=torch.int64, device=dev)
            best_ref = torch.zeros(2, dtype=torch.int64, device=dev)
            h.sweep_dev(count, best_ref, first_code=first, tel_out=tel)
            h.sync()
            best = torch.full((2,), -7, dtype=torch.int64, device=dev)
            kv.argmin_static_dev(tel, best, index_base=first)
            torch.cuda.synchronize()
            assert best.tolist() == best_ref.tolist(), call
            t = tel.cpu().numpy()
            assert best[0].item() == t.min() and best[1].item() == first + int(np.argmin(t))
        # equal TELs everywhere: the lowest index wins
        flat = torch.full((5000,), 42, dtype=torch.int64, device=dev)
        kv.argmin_static_dev(flat, best, index_base=10)
        torch.cuda.synchronize()
        assert best.tolist() == [42, 10]


def test_static_argmin_rejects_bad_sizes():
    import torch
    from paper_2508_06133_b200 import binding as kv

    dev = torch.device("cuda", torch.cuda.current_device())
    tel = torch.zeros(8, dtype=torch.int64, device=dev)
    best = torch.zeros(2, dtype=torch.int64, device=dev)
    with pytest.raises(kv.SchedError) as e:
        kv.argmin_static_dev(tel, best, count=(1 << 26) + 1)
    assert e.value.code == kv.E_UNSUPPORTED
    assert b"exceeds the fixed limit" in kv.load().sched_last_cuda_error()
    with pytest.raises(kv.SchedError) as e:
        kv.argmin_static_dev(tel, best, count=0)
    assert e.value.code == kv.E_INVAL
