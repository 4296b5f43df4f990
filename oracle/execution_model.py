"""Oracle for the paper's trace-completion-time formula (Sec. 5.1, Eq. "ttotal").

TEST INFRASTRUCTURE ONLY; shares no code with the package.  The equation written
out term by term over explicit lists, 1-based like the paper:

    T_total = t_sched(1) + t_serve(1) + sum_{i=2}^{N} [ t_stale(i) + t_reconfig(i) + t_serve(i) ]

Pin (tests/test_oracle_pins.py): the three rows of the paper's table of example
artifact feedback (tests/golden/table_artifact_feedback.txt): the accumulated
costs it prints add up to the T_total it prints.
"""


def t_total(t_sched, t_stale, t_reconfig, t_serve):
    """Lists indexed by interval, entry 0 = interval 1.  t_stale[0] and t_reconfig[0] do not exist
    in the model (the first interval is a cold start) and are ignored."""
    n = len(t_serve)
    if n == 0:
        return 0.0
    total = t_sched[0] + t_serve[0]
    i = 2
    while i <= n:
        total += t_stale[i - 1] + t_reconfig[i - 1] + t_serve[i - 1]
        i += 1
    return total
