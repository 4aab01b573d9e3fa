"""Host logic of the multi-task manager and its asynchronous loop (Algorithm 1), without a GPU: version gating (one
rollout per committed version, every update on-policy), FIFO hand-off, KV-budget admission in arrival order."""
import threading
import time

import pytest

from paper_2605_08527_b200 import manager as M


def test_kv_cache_estimate_is_keys_plus_values_of_every_layer_and_position():
    # 7B-shaped: 32 layers, 32 KV heads of 128, bf16: 0.5 MiB per position
    assert M.kv_cache_bytes(1, 1, 32, 32, 128) == 2 * 32 * 32 * 128 * 2
    assert M.kv_cache_bytes(8, 4096, 32, 32, 128) == 8 * 4096 * 524288


def test_admission_respects_the_budget_in_arrival_order():
    m = M.MultiTaskManager(kv_budget_bytes=100)
    assert m.add_task(0, 60) is True
    assert m.add_task(1, 50) is False           # 110 > 100: waits
    assert m.add_task(2, 10) is False           # would fit, but does not overtake task 1
    assert m.next_policy(1) is None and m.next_policy(2) is None and m.next_policy(0) == 0
    m.retire_task(0)
    assert m.tasks[1].admitted and m.tasks[2].admitted and m.kv_in_use() == 60
    big = M.MultiTaskManager(kv_budget_bytes=10)
    assert big.add_task(7, 1000) is True        # a task larger than the budget still runs when nothing else does


def test_version_gating_and_off_policy_updates():
    m = M.MultiTaskManager(kv_budget_bytes=1 << 40)
    m.add_task(3, 1)
    assert m.next_policy(3) == 0
    assert m.next_policy(3) is None             # version 0 was already handed out: wait for the commit
    m.enqueue(3, "tau0", 0)
    task, tau, v = m.pop()
    assert (task, tau, v) == (3, "tau0", 0)
    with pytest.raises(RuntimeError):
        m.commit(3, 1)                          # the policy is at version 0
    assert m.commit(3, 0) == 1
    assert m.next_policy(3) == 1
    with pytest.raises(RuntimeError):
        m.commit(3, 0)                          # a second update from the stale rollout
    assert m.pop(block=False) is None


def test_loop_runs_every_task_to_its_last_version_on_policy_and_in_fifo_order():
    m = M.MultiTaskManager(kv_budget_bytes=250)
    tasks = list(range(6))
    for t in tasks:
        m.add_task(t, 100)                      # two tasks fit at a time
    seen, trained, concurrent, peak = [], [], [0], [0]
    lock = threading.Lock()

    def rollout(task, version, device_lock):
        with lock:
            concurrent[0] += 1
            peak[0] = max(peak[0], concurrent[0])
        time.sleep(0.002 * (1 + task % 3))      # rollouts of different lengths
        with lock:
            concurrent[0] -= 1
            seen.append((task, version))
        return ("tau", task, version)

    def update(task, tau, version, device_lock):
        assert tau == ("tau", task, version)
        assert m.tasks[task].version == version  # on-policy
        with device_lock:
            trained.append((task, version))

    M.run_loop(m, tasks, 4, rollout, update)
    assert sorted(seen) == [(t, v) for t in tasks for v in range(4)]
    assert sorted(trained) == sorted(seen)
    for t in tasks:
        assert [v for tt, v in trained if tt == t] == [0, 1, 2, 3]      # in order, each exactly once
        assert m.tasks[t].version == 4 and m.tasks[t].updates == 4 and m.tasks[t].rollouts == 4
    assert peak[0] <= 2                          # never more rollouts in flight than the budget admits
    # the queue is first in, first out: updates follow the order in which rollouts were enqueued
    enq = [(t, v) for (ev, t, v) in m.log if ev == "rollout"]
    assert len(enq) == 24 and len([e for e in m.log if e[0] == "commit"]) == 24


def test_an_exception_in_a_worker_stops_the_loop_and_is_raised():
    m = M.MultiTaskManager(kv_budget_bytes=1 << 30)
    m.add_task(0, 1)

    def bad_update(task, tau, version, device_lock):
        raise ValueError("boom")

    with pytest.raises(ValueError):
        M.run_loop(m, [0], 2, lambda t, v, l: None, bad_update)
