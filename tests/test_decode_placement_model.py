"""Host-side model of the run-time placement of the <= 16-token decode launches (sched_enter in
csrc/w4a8_linear_splitn.cuh): a launch has more candidate CTAs than it needs workers; every
candidate (1) reads the count of issued worker indices, (2) takes a start number and counts itself
in on its SM, (3) decides, (4) draws an index if it wants to work.  The steps of different
candidates interleave freely.  Checked over ALL interleavings of small cases: every worker index is
issued exactly once -- a missing one would leave a tile of the layer uncomputed.  The same search
over the order that reads the count AFTER taking the start number finds the interleaving in which
an index goes missing, which is why the kernel reads first (with an acquire load)."""
import itertools

import pytest


def _explore(workers, sm_of, read_first):
    """Depth-first search over all interleavings; returns the set of final `issued` counts and the
    worst number of indices drawn beyond `workers`."""
    n = len(sm_of)
    steps = ("read", "start", "draw") if read_first else ("start", "read", "draw")
    seen = set()
    finals = set()

    def run(state):
        if state in seen:
            return
        seen.add(state)
        pcs, issued, started, on_sm, regs = state
        if all(pc == 3 for pc in pcs):
            finals.add(min(issued, workers))
            return
        for k in range(n):
            pc = pcs[k]
            if pc == 3:
                continue
            i_seen, c, first = regs[k]
            n_issued, n_started, n_on = issued, started, on_sm
            op = steps[pc]
            if op == "read":
                i_seen = issued
            elif op == "start":
                c = started
                n_started = started + 1
                first = on_sm[sm_of[k]] == 0
                lst = list(on_sm)
                lst[sm_of[k]] += 1
                n_on = tuple(lst)
            else:
                want = first or (i_seen < workers and workers - i_seen >= n - c)
                if want:
                    n_issued = issued + 1      # (an index >= workers makes the candidate retire after all)
            nregs = regs[:k] + ((i_seen, c, first),) + regs[k + 1:]
            npcs = pcs[:k] + (pc + 1,) + pcs[k + 1:]
            run((npcs, n_issued, n_started, n_on, nregs))

    nsm = max(sm_of) + 1
    run(((0,) * n, 0, 0, (0,) * nsm, ((0, 0, False),) * n))
    return finals


@pytest.mark.parametrize("workers,sm_of", [
    (2, (0, 0, 1, 1)),        # two SMs, two candidates each: the normal case
    (2, (0, 0, 0, 1)),        # three candidates land on one SM
    (2, (0, 0, 0, 0)),        # all on one SM: second workers are forced
    (3, (0, 0, 1, 1)),        # more workers than SMs with room
    (1, (0, 1, 1)),
    (3, (0, 0, 0, 1, 1)),
])
def test_every_worker_index_is_issued_in_every_interleaving(workers, sm_of):
    assert _explore(workers, sm_of, read_first=True) == {workers}


def test_reading_the_count_after_the_start_number_can_lose_an_index():
    # the order the kernel does NOT use: some interleaving of some small case ends with fewer
    # indices issued than there are workers
    lost = False
    for workers, sm_of in itertools.product((1, 2, 3), ((0, 0, 0), (0, 0, 0, 0), (0, 0, 1, 1), (0, 0, 0, 1))):
        if workers > len(sm_of):
            continue
        if _explore(workers, sm_of, read_first=False) != {workers}:
            lost = True
    assert lost
