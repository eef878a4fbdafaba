"""Batch scheduler (Section 5.2, Section 6.1) against a plain Python model of its rules: API type by
oldest eligible call, vertical batching of head-of-queue runs that stops at a write-write conflict,
horizontal batching across queues, priority order, truncation from the tail."""
import random

import paper_2510_24051_b200 as pie

FORWARD, EMBED, SAMPLE = 0, 1, 2


class Model:
    """Reference scheduler: the rules written out with lists."""

    def __init__(self, max_batch):
        self.max_batch, self.queues, self.prio = max_batch, [], []

    def create_queue(self, prio):
        self.queues.append([])
        self.prio.append(prio)
        return len(self.queues) - 1

    def submit(self, q, typ, writes, t, tag):
        self.queues[q].append((typ, set(writes), t, tag))

    def next_batch(self):
        oldest = {}
        for calls in self.queues:
            if not calls:
                continue
            typ = calls[0][0]
            for c in calls:
                if c[0] != typ:
                    break
                oldest[typ] = min(oldest.get(typ, c[2]), c[2])
        if not oldest:
            return -1, [], []
        typ = min(sorted(oldest), key=lambda t: oldest[t])
        order = sorted((q for q, calls in enumerate(self.queues) if calls and calls[0][0] == typ),
                       key=lambda q: (-self.prio[q], q))
        written, tags, qs = set(), [], []
        for q in order:
            calls = self.queues[q]
            while calls and calls[0][0] == typ and len(tags) < self.max_batch:
                if calls[0][1] & written:
                    break
                written |= calls[0][1]
                tags.append(calls[0][3])
                qs.append(q)
                calls.pop(0)
            if len(tags) >= self.max_batch:
                break
        return typ, tags, qs


def test_figure_example_forward_batch_of_three_or_embed_batch_of_two():
    s = pie.pie_sched_create(64)
    q = [pie.pie_sched_create_queue(s) for _ in range(4)]
    pie.pie_sched_submit(s, q[0], FORWARD, [10], 100, 1)
    pie.pie_sched_submit(s, q[0], FORWARD, [11], 101, 2)        # vertical: same queue, different page
    pie.pie_sched_submit(s, q[1], FORWARD, [20], 102, 3)        # horizontal
    pie.pie_sched_submit(s, q[1], EMBED, [], 103, 4)            # behind a forward in its queue: not eligible yet
    pie.pie_sched_submit(s, q[2], EMBED, [], 104, 5)
    pie.pie_sched_submit(s, q[3], EMBED, [], 105, 6)
    assert pie.pie_sched_pending(s) == 6
    assert pie.pie_sched_next_batch(s) == (FORWARD, [1, 2, 3], [q[0], q[0], q[1]])   # oldest call is a forward
    assert pie.pie_sched_next_batch(s) == (EMBED, [4, 5, 6], [q[1], q[2], q[3]])
    assert pie.pie_sched_next_batch(s) == (-1, [], [])
    pie.pie_sched_destroy(s)


def test_vertical_conflict_priority_and_truncation():
    s = pie.pie_sched_create(3)
    lo = pie.pie_sched_create_queue(s, priority=0)
    hi = pie.pie_sched_create_queue(s, priority=5)
    pie.pie_sched_submit(s, lo, FORWARD, [1], 10, 100)
    pie.pie_sched_submit(s, lo, FORWARD, [1], 11, 101)          # writes the same KvPage as the call before it
    pie.pie_sched_submit(s, lo, FORWARD, [2], 12, 102)
    pie.pie_sched_submit(s, hi, FORWARD, [7], 20, 200)
    pie.pie_sched_submit(s, hi, FORWARD, [8], 21, 201)
    # higher-priority queue first; the low queue contributes only up to its conflict; limit 3
    assert pie.pie_sched_next_batch(s) == (FORWARD, [200, 201, 100], [hi, hi, lo])
    assert pie.pie_sched_next_batch(s) == (FORWARD, [101, 102], [lo, lo])
    pie.pie_sched_set_queue_priority(s, lo, 9)
    pie.pie_sched_submit(s, hi, FORWARD, [3], 30, 202)
    pie.pie_sched_submit(s, lo, FORWARD, [4], 31, 103)
    assert pie.pie_sched_next_batch(s, cap=1) == (FORWARD, [103], [lo])   # caller's cap truncates too
    assert pie.pie_sched_next_batch(s) == (FORWARD, [202], [hi])
    pie.pie_sched_destroy(s)


def test_random_traffic_matches_model():
    rng = random.Random(7)
    for trial in range(30):
        max_batch = rng.choice([1, 2, 5, 64])
        s, m = pie.pie_sched_create(max_batch), Model(max_batch)
        nq = rng.randint(1, 6)
        for _ in range(nq):
            p = rng.randint(0, 3)
            assert pie.pie_sched_create_queue(s, p) == m.create_queue(p)
        t, tag = 0, 0
        for step in range(60):
            for _ in range(rng.randint(0, 5)):
                q, typ = rng.randrange(nq), rng.choice([FORWARD, FORWARD, EMBED, SAMPLE])
                writes = [rng.randrange(6) for _ in range(rng.randint(0, 2))] if typ == FORWARD else []
                t += rng.randint(0, 3)
                tag += 1
                pie.pie_sched_submit(s, q, typ, writes, t, tag)
                m.submit(q, typ, writes, t, tag)
            if rng.random() < 0.6:                                # "GPU idle": form a batch
                assert pie.pie_sched_next_batch(s) == m.next_batch()
        while True:                                               # drain
            got = pie.pie_sched_next_batch(s)
            assert got == m.next_batch()
            if got[0] < 0:
                break
        assert pie.pie_sched_pending(s) == 0
        pie.pie_sched_destroy(s)
