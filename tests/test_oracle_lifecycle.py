"""The lifecycle model against Algorithm 1 and Fig. lifecycle: allowed transitions, retention of
every logical page, per-format free lists, failure codes."""
import random

import pytest

from oracle.lifecycle import (ANCHOR, FMT_FP8, FMT_TQ3, RECENT, STALE, LifecycleError, PoolModel)


def test_append_opens_a_page_every_16_tokens_and_publishes_recent():
    pool = PoolModel(4, 4)
    s = pool.new_seq()
    opened = [s.append() for _ in range(33)]
    assert [o[2] for o in opened].count(True) == 3
    assert [o[1] for o in opened[:17]] == list(range(16)) + [0]
    assert [t for t, _ in s.pages] == [RECENT] * 3 and s.len == 33
    pool.check_invariants()


def test_transitions_of_the_lifecycle_graph():
    pool = PoolModel(8, 8)
    s = pool.new_seq()
    for _ in range(16 * 3 + 2):
        s.append()
    s.protect(0)                                   # Recent -> Anchor
    assert s.pages[0][0] == ANCHOR
    src, dst = s.demote(1)                         # Recent -> Stale (age)
    assert s.pages[1] == (STALE, dst)
    # the source is retiring: not mapped, not free, and the next page a request opens is another one
    assert (FMT_FP8, src) in pool.retiring and src not in pool.free[FMT_FP8]
    other = pool.new_seq()
    assert other.append()[0] != src
    with pytest.raises(LifecycleError) as e:
        other.release(FMT_FP8, src)                # only the owning request releases it
    assert e.value.code == "MKV_E_STATE"
    s.release(FMT_FP8, src)
    assert src in pool.free[FMT_FP8] and not pool.retiring
    with pytest.raises(LifecycleError):
        s.release(FMT_FP8, src)                    # once
    other.finish()
    s.demote(0)                                    # Anchor -> Stale (demote)
    with pytest.raises(LifecycleError) as e:
        s.protect(0)                               # Stale cannot be tagged; it must be promoted
    assert e.value.code == "MKV_E_STATE"
    src, dst = s.promote(0)                        # Stale -> Anchor through a new FP8 page
    assert s.pages[0] == (ANCHOR, dst) and (FMT_TQ3, src) in pool.retiring and src not in pool.free[FMT_TQ3]
    with pytest.raises(LifecycleError):
        s.demote(3)                                # the open, partial page never becomes TQ3
    with pytest.raises(LifecycleError):
        s.demote(1)                                # already Stale
    with pytest.raises(LifecycleError) as e:
        s.demote(9)
    assert e.value.code == "MKV_E_BOUNDS"
    pool.check_invariants()
    assert len(s.pages) == 4                       # nothing was dropped
    s.finish()
    assert len(pool.free[FMT_FP8]) == 8 and len(pool.free[FMT_TQ3]) == 8 and not pool.owner


def test_exhaustion_reports_the_arena_and_changes_nothing():
    pool = PoolModel(2, 1)
    s = pool.new_seq()
    for _ in range(32):
        s.append()
    with pytest.raises(LifecycleError) as e:
        s.append()
    assert e.value.code == "MKV_E_OOM_FP8" and s.len == 32
    s.demote(0)
    with pytest.raises(LifecycleError) as e:
        s.demote(1)
    assert e.value.code == "MKV_E_OOM_TQ3" and s.pages[1][0] == RECENT
    pool.check_invariants()


def test_age_demotes_exactly_the_full_recent_pages_outside_the_window():
    pool = PoolModel(64, 64)
    s = pool.new_seq()
    for _ in range(16 * 10 + 7):
        s.append()
    s.protect(2)
    moved = s.age(recent_tokens=40)      # window starts at token 127 -> page 7
    assert [m[0] for m in moved] == [0, 1, 3, 4, 5, 6]
    assert [t for t, _ in s.pages] == [STALE, STALE, ANCHOR, STALE, STALE, STALE, STALE, RECENT, RECENT, RECENT, RECENT]
    pool.check_invariants()


def test_random_walk_keeps_every_invariant():
    rnd = random.Random(0)
    pool = PoolModel(40, 40)
    seqs = []
    for step in range(4000):
        r = rnd.random()
        try:
            if r < 0.02 or not seqs:
                seqs.append(pool.new_seq())
            elif r < 0.70:
                rnd.choice(seqs).append()
            elif r < 0.80:
                s = rnd.choice(seqs)
                if s.pages:
                    s.demote(rnd.randrange(len(s.pages)))
            elif r < 0.86:
                s = rnd.choice(seqs)
                if s.pages:
                    s.promote(rnd.randrange(len(s.pages)))
            elif r < 0.92:
                s = rnd.choice(seqs)
                if s.pages:
                    s.protect(rnd.randrange(len(s.pages)))
            elif r < 0.94:
                rnd.choice(seqs).age(rnd.choice([16, 48, 100]))
            elif r < 0.96:
                if pool.retiring:                  # the stream point of some conversion has passed
                    (fmt, pid), h = rnd.choice(sorted(pool.retiring.items()))
                    pool.seqs[h].release(fmt, pid)
            else:
                s = seqs.pop(rnd.randrange(len(seqs)))
                s.finish()
        except LifecycleError:
            pass
        pool.check_invariants()
    used, tiers = pool.stats()
    assert used[FMT_FP8] == tiers[RECENT] + tiers[ANCHOR] and used[FMT_TQ3] == tiers[STALE]
