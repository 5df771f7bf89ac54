"""Host logic of the recurrent kernel's operand ring, checked without a GPU.

One producer thread fills the ring stages and several MMA issuer threads drain them; an mbarrier wait only
sees the parity of a stage's round, so the schedule must guarantee that (a) within a phase every stage is used
by exactly one issuer, (b) that issuer meets the rounds of its stages in order, and (c) the per-stage round
counters carried from phase to phase count exactly the fills.  The test replays the producer's and the issuers'
loops as the kernel runs them, over every stage / issuer / chunk count the launcher can choose, for several
phases in a row.
"""
import itertools

import pytest

import paper_2101_05453_b200 as qlstm
from paper_2101_05453_b200.binding import QlstmError, ring_plan


def producer_sequence(pl, contiguous):
    """(owner, chunk-in-tile, stage, local round) in the order the producer issues the copies."""
    kk, rr, seq = [0] * 4, [0] * 4, []
    for j in range(pl["n_max"]):
        for o in range(4):
            if o >= pl["n_own"] or j >= pl["n_chunks"][o]:
                continue
            c = j if contiguous else o + j * pl["n_own"]
            stage = o + pl["n_own"] * kk[o]
            seq.append((o, c, stage, rr[o]))
            kk[o] += 1
            if kk[o] == pl["cnt"][o]:
                kk[o] = 0
                rr[o] += 1
    return seq


def issuer_sequence(pl, me, contiguous):
    kk, rr, seq = 0, 0, []
    for j in range(pl["n_chunks"][me]):
        c = j if contiguous else me + j * pl["n_own"]
        seq.append((me, c, me + pl["n_own"] * kk, rr))
        kk += 1
        if kk == pl["cnt"][me]:
            kk, rr = 0, rr + 1
    return seq


CASES = [(stages, n_own, contiguous, n)
         for stages in (1, 2, 3, 4) for n_own in (1, 2, 3, 4) if n_own <= stages
         for contiguous in (True, False) for n in (0, 1, 2, 3, 5, 8, 16, 17)]


@pytest.mark.parametrize("stages,n_own,contiguous,n", CASES)
def test_plan_invariants(stages, n_own, contiguous, n):
    pl = ring_plan(stages, n_own, contiguous, chunks_per_tile=n, chunks_total=n)
    assert pl["n_own"] == n_own
    prod = producer_sequence(pl, contiguous)
    # every chunk exactly once: one tile of n chunks per owner, or n chunks shared by the owners
    if contiguous:
        assert sorted((o, c) for o, c, _, _ in prod) == [(o, c) for o in range(n_own) for c in range(n)]
    else:
        assert sorted(c for _, c, _, _ in prod) == list(range(n))
        assert all(c % n_own == o for o, c, _, _ in prod)
    # a stage has one owner, lies inside the ring, and its fills are counted in uses[]
    owner_of, fills = {}, [0] * 4
    for o, _, stage, _ in prod:
        assert 0 <= stage < stages
        assert owner_of.setdefault(stage, o) == o
        fills[stage] += 1
    assert fills == pl["uses"]
    # each issuer sees exactly the producer's chunks of its stages, same stage and round, in the same order,
    # and the rounds of one stage come in order 0, 1, 2, ...
    for me in range(n_own):
        mine = issuer_sequence(pl, me, contiguous)
        assert mine == [e for e in prod if e[0] == me]
        per_stage = {}
        for _, _, stage, rnd in mine:
            assert rnd == per_stage.get(stage, 0)
            per_stage[stage] = rnd + 1


def test_round_counters_carry_over_alternating_phases():
    """Phases alternate between the two matmuls with different owner counts: a stage may change owner between
    phases, and the parity the next phase expects must be the one the counters predict."""
    for stages, own_a, own_c, per, total in itertools.product((2, 3, 4), (1, 2), (1, 2, 3, 4), (3, 5), (8, 16)):
        if own_a > stages or own_c > stages:
            continue
        plan_a = ring_plan(stages, own_a, True, chunks_per_tile=per)
        plan_c = ring_plan(stages, own_c, False, chunks_total=total)
        rounds, completed = [0] * 4, [0] * 4          # counters as the kernel keeps them / fills that really happened
        for step in range(5):
            for pl, contiguous in ((plan_a, True), (plan_c, False)):
                for o, _, stage, rnd in producer_sequence(pl, contiguous):
                    assert rounds[stage] + rnd == completed[stage]      # the fill the waiter expects is the next one
                    completed[stage] += 1
                rounds = [r + u for r, u in zip(rounds, pl["uses"])]
                assert rounds == completed


def test_rejects_more_owners_than_stages():
    with pytest.raises(QlstmError):
        ring_plan(2, 3, False, chunks_total=8)
    with pytest.raises(QlstmError):
        ring_plan(5, 1, True, chunks_per_tile=3)
