"""Host-only toy of the multi-task manager and its asynchronous loop (Methods: Multi-Task Manager, KV-Cache-Aware
Scheduling, Asynchronous Execution, Multi-LoRA Rollout with Single-Task Training; Algorithm 1).

Per task the manager keeps the committed policy version v (the adapter parameters and the optimizer state themselves
live wherever the caller keeps them: in the pooled adapter store and in its fp32 masters / moments), whether that
version has already been handed to the rollout engine, and an estimate of the task's KV-cache footprint.  A global
FIFO pairs every rollout with the version that generated it.  Rollout runs for all admitted tasks in parallel
(one host thread per task here), training takes one queued rollout at a time; a task's next rollout waits until the
update that consumes its previous one has been committed, so every update is on-policy: the rollout of version v is
consumed by exactly the update v -> v + 1.

Nothing in this module touches the GPU.  The rollout and update work is whatever callables the caller passes; when
they call the layer (marlaas_lora_forward / _backward / marlaas_adapter_pool_adamw_commit) on one pool they must
serialise those calls themselves (the `device_lock` handed to them), as the C ABI asks.
"""
from __future__ import annotations

import collections
import dataclasses
import threading
from typing import Any, Callable, Deque, Dict, List, Optional, Tuple


def kv_cache_bytes(batch: int, gen_len: int, n_layers: int, n_kv_heads: int, head_dim: int, bytes_per_value: int = 2) -> int:
    """KV-cache footprint of one task's rollout batch: keys and values of every layer for every generated position
    (KV-Cache-Aware Scheduling: estimated from generation length, batch size and model configuration)."""
    return 2 * n_layers * n_kv_heads * head_dim * bytes_per_value * gen_len * batch


@dataclasses.dataclass
class TaskState:
    task: int
    version: int = 0                    # committed policy version v
    handed_out: bool = False            # version v has already been given to the rollout engine
    kv_bytes: int = 0
    admitted: bool = False
    rollouts: int = 0
    updates: int = 0


class MultiTaskManager:
    """Versioned per-task state, the KV-budget admission test and the global FIFO of (task, rollout, version)."""

    def __init__(self, kv_budget_bytes: int):
        self.kv_budget = int(kv_budget_bytes)
        self.tasks: Dict[int, TaskState] = {}
        self.waiting: Deque[int] = collections.deque()          # tasks not admitted yet, in arrival order
        self.q_buffer: Deque[Tuple[int, Any, int]] = collections.deque()
        self.cv = threading.Condition()
        self.stopped = False
        self.log: List[Tuple[str, int, int]] = []               # (event, task, version), in the order they happened

    # ---- admission -------------------------------------------------------------------------------------------
    def kv_in_use(self) -> int:
        return sum(t.kv_bytes for t in self.tasks.values() if t.admitted)

    def add_task(self, task: int, kv_bytes: int) -> bool:
        """Registers a task at version 0; it is admitted at once if the aggregate KV estimate stays within the budget,
        otherwise it waits (first come, first served) until retire_task frees room.  Returns whether it was admitted."""
        with self.cv:
            assert task not in self.tasks
            self.tasks[task] = TaskState(task, kv_bytes=int(kv_bytes))
            self.waiting.append(task)
            self._admit_waiting()
            self.cv.notify_all()
            return self.tasks[task].admitted

    def retire_task(self, task: int) -> None:
        with self.cv:
            self.tasks[task].admitted = False
            self.tasks[task].kv_bytes = 0
            self._admit_waiting()
            self.cv.notify_all()

    def _admit_waiting(self) -> None:
        while self.waiting:
            t = self.tasks[self.waiting[0]]
            if self.kv_in_use() + t.kv_bytes > self.kv_budget and self.kv_in_use() > 0:
                break                                           # head of the line does not fit: nobody overtakes it
            t.admitted = True
            self.waiting.popleft()
            self.log.append(("admit", t.task, t.version))

    # ---- Algorithm 1 ------------------------------------------------------------------------------------------
    def next_policy(self, task: int) -> Optional[int]:
        """The next policy version of the task that no rollout has consumed yet, or None."""
        with self.cv:
            t = self.tasks[task]
            if not t.admitted or t.handed_out:
                return None
            t.handed_out = True
            self.log.append(("rollout", task, t.version))
            return t.version

    def wait_next_policy(self, task: int) -> Optional[int]:
        """Blocks until next_policy(task) exists (None once the manager is stopped)."""
        with self.cv:
            while not self.stopped:
                t = self.tasks[task]
                if t.admitted and not t.handed_out:
                    t.handed_out = True
                    self.log.append(("rollout", task, t.version))
                    return t.version
                self.cv.wait(timeout=0.05)
            return None

    def enqueue(self, task: int, rollout: Any, version: int) -> None:
        with self.cv:
            self.tasks[task].rollouts += 1
            self.q_buffer.append((task, rollout, version))
            self.cv.notify_all()

    def pop(self, block: bool = True) -> Optional[Tuple[int, Any, int]]:
        with self.cv:
            while not self.q_buffer:
                if not block or self.stopped:
                    return None
                self.cv.wait(timeout=0.05)
            return self.q_buffer.popleft()

    def commit(self, task: int, from_version: int) -> int:
        """The update that consumed the rollout of `from_version` is done: version from_version + 1 becomes the task's
        policy and is eligible for rollout.  An update from any other version than the committed one is off-policy."""
        with self.cv:
            t = self.tasks[task]
            if from_version != t.version or not t.handed_out:
                raise RuntimeError(f"off-policy update of task {task}: rollout of version {from_version}, policy at {t.version}")
            t.version += 1
            t.handed_out = False
            t.updates += 1
            self.log.append(("commit", task, t.version))
            self.cv.notify_all()
            return t.version

    def stop(self) -> None:
        with self.cv:
            self.stopped = True
            self.cv.notify_all()


def run_loop(manager: MultiTaskManager, tasks: List[int], versions_per_task: int,
             rollout_fn: Callable[[int, int, threading.Lock], Any], update_fn: Callable[[int, Any, int, threading.Lock], None]) -> None:
    """Algorithm 1 on host threads: one rollout thread per task, one training thread.  rollout_fn(task, version,
    device_lock) returns the rollout; update_fn(task, rollout, version, device_lock) performs the policy update and the
    commit of the new parameters (into the adapter store); the manager's own commit follows it.  Every task stops after
    `versions_per_task` updates."""
    device_lock = threading.Lock()
    errors: List[BaseException] = []

    def rollout_worker(task: int) -> None:
        try:
            for _ in range(versions_per_task):
                v = manager.wait_next_policy(task)
                if v is None:
                    return
                manager.enqueue(task, rollout_fn(task, v, device_lock), v)
        except BaseException as e:  # noqa: BLE001
            errors.append(e)
            manager.stop()

    def trainer() -> None:
        try:
            for _ in range(versions_per_task * len(tasks)):
                item = manager.pop()
                if item is None:
                    return
                task, rollout, v = item
                update_fn(task, rollout, v, device_lock)
                manager.commit(task, v)
                if manager.tasks[task].updates == versions_per_task:
                    manager.retire_task(task)
        except BaseException as e:  # noqa: BLE001
            errors.append(e)
            manager.stop()

    threads = [threading.Thread(target=rollout_worker, args=(t,), daemon=True) for t in tasks]
    threads.append(threading.Thread(target=trainer, daemon=True))
    for th in threads:
        th.start()
    for th in threads:
        th.join(timeout=120)
    manager.stop()
    if errors:
        raise errors[0]
    if any(th.is_alive() for th in threads):
        raise RuntimeError("the loop did not finish")
