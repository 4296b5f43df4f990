"""The paper's execution model (Sec. 5.1, Eq. "ttotal") applied to measured serving iterations.

A trace is served in rescheduling intervals.  The first is a cold start: the
policy computes a plan (t_sched) and the system serves under it (t_serve).
Every later interval, opened when ``should_reschedule`` fires, has three
phases: the old plan keeps serving while the new one is computed (t_stale),
the system moves to the new plan (t_reconfig), and it serves under the new plan
(t_serve).  The trace completion time is

    T_total = t_sched(1) + t_serve(1) + sum_{i >= 2} [t_stale(i) + t_reconfig(i) + t_serve(i)]

and the evaluator's artifact feedback (Sec. 5.3, table "artifact feedback") is
the number of reschedulings with the three accumulated costs.

Here the serving cost of an interval is not simulated: it is the measured device
time of the interval's serving iterations on this library (append + attention
of one layer), so fixed scheduling policies (token budget, prefill chunk size)
can be compared on the workload-shift trace by the quantity the paper's search
minimises.  Host-side arithmetic only.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Iterable, List, Sequence


@dataclass
class Interval:
    """Costs of one rescheduling interval, in seconds.  ``t_sched`` counts for the first interval
    only (later scheduling time is on the timeline as ``t_stale``); ``t_stale`` and ``t_reconfig``
    count for intervals after the first."""
    t_sched: float = 0.0
    t_stale: float = 0.0
    t_reconfig: float = 0.0
    t_serve: float = 0.0


def total_time(intervals: Sequence[Interval]) -> float:
    """Eq. "ttotal"."""
    if not intervals:
        return 0.0
    first, rest = intervals[0], intervals[1:]
    return first.t_sched + first.t_serve + sum(iv.t_stale + iv.t_reconfig + iv.t_serve for iv in rest)


def artifact_feedback(intervals: Sequence[Interval]) -> Dict[str, float]:
    """The evaluator's cost breakdown: reschedulings (intervals after the cold start), accumulated
    stale, reconfiguration and serving cost, and T_total."""
    rest = intervals[1:]
    return {"N": max(len(intervals) - 1, 0),
            "sum_t_stale": sum(iv.t_stale for iv in rest),
            "sum_t_reconfig": sum(iv.t_reconfig for iv in rest),
            "sum_t_serve": sum(iv.t_serve for iv in intervals),
            "T_total": total_time(intervals)}


def intervals_from_iterations(iteration_seconds: Iterable[float], reschedule_at: Sequence[int] = (),
                              t_sched_first: float = 0.0, t_stale: Sequence[float] = (),
                              t_reconfig: Sequence[float] = ()) -> List[Interval]:
    """Groups measured per-iteration serving times into intervals.  ``reschedule_at`` lists the
    iteration indices at which a new interval opens (increasing); interval i >= 2 carries
    ``t_stale[i-2]`` and ``t_reconfig[i-2]``.  A fixed policy never reschedules: one interval."""
    times = list(iteration_seconds)
    cuts = [0] + list(reschedule_at) + [len(times)]
    if any(b < a for a, b in zip(cuts[:-1], cuts[1:])) or (reschedule_at and reschedule_at[0] <= 0):
        raise ValueError("reschedule_at must be increasing iteration indices inside the trace")
    out = []
    for i, (a, b) in enumerate(zip(cuts[:-1], cuts[1:])):
        iv = Interval(t_serve=float(sum(times[a:b])))
        if i == 0:
            iv.t_sched = float(t_sched_first)
        else:
            iv.t_stale = float(t_stale[i - 1]) if i - 1 < len(t_stale) else 0.0
            iv.t_reconfig = float(t_reconfig[i - 1]) if i - 1 < len(t_reconfig) else 0.0
        out.append(iv)
    return out
