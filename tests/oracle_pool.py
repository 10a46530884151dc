"""Oracle runs in worker processes (started with spawn: the parent may hold a CUDA context).

A task names an instance of a workload by its index; the worker regenerates that instance from the seed, so that
nothing large crosses the process boundary.
"""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def solve_instance(task):
    """task = (workload as a dict of its fields, instance index, objective) -> (instance, objective, wait, barrier, idx)."""
    import numpy as np

    import oracle as o
    import zl_inputs as zi
    fields, b, objective = task
    w = zi.Workload(**fields)
    ts = zi.generate(w, B=1, first_instance=b)
    wait, barrier, idx = o.sweep_window(ts[0], objective)
    return b, objective, int(wait), int(barrier), np.asarray(idx, dtype=np.int32)


def solve_all(w, instances, objectives, processes=None):
    """The oracle on the given instances of workload w, for each objective; a dict keyed by (instance, objective)."""
    import dataclasses
    import multiprocessing as mp
    fields = dataclasses.asdict(w)
    tasks = [(fields, b, obj) for obj in objectives for b in instances]
    processes = processes or max(1, min(len(tasks), (os.cpu_count() or 2) - 1, 16))
    if processes == 1:
        results = [solve_instance(t) for t in tasks]
    else:
        with mp.get_context("spawn").Pool(processes) as pool:
            results = pool.map(solve_instance, tasks, chunksize=1)
    return {(b, obj): (wt, bar, idx) for b, obj, wt, bar, idx in results}
