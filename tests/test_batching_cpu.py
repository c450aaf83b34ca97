"""The job queue of continuous batching (Appendix A.11 / A.12) with a stand-in for the model: requests join and leave
between steps, every request keeps its own cache slot and consecutive positions, one micro-batch per step, and the
tokens of a request do not depend on who shared its steps."""
import numpy as np
import pytest

from paper_2504_08791_b200.batching import JobQueue


class FakeExecutor:
    """A 'model' whose next token is a hash of all tokens the request has fed so far.  It keeps one history per cache
    slot, indexed by position, exactly as the caches of the real executor are, and checks the calling discipline."""

    def __init__(self, max_batch=4, kv_capacity=64):
        self.max_batch = max_batch
        self.kv_capacity = kv_capacity
        self.cache = {}
        self.calls = []

    @staticmethod
    def next_token(history):
        h = 7
        for t in history:
            h = (h * 1_000_003 + int(t) + 1) % 2_147_483_647
        return h % 5000

    def step(self, tokens, slots, positions):
        assert 1 <= len(tokens) <= self.max_batch
        assert len(set(slots)) == len(slots), "a cache slot appears once per micro-batch"
        out = []
        for tok, slot, pos in zip(tokens, slots, positions):
            hist = self.cache.setdefault(slot, [])
            assert 0 <= pos <= len(hist) and pos < self.kv_capacity
            del hist[pos:]                      # a new holder of the slot starts at 0 and overwrites
            hist.append(tok)
            out.append(self.next_token(hist))
        self.calls.append((list(tokens), list(slots), list(positions)))
        return np.asarray(out, np.int32)


def alone(prompt, n_new, eos=None):
    hist, out = list(prompt), []
    while len(out) < n_new:
        out.append(FakeExecutor.next_token(hist))
        if eos is not None and out[-1] == eos:
            break
        hist.append(out[-1])
    return out


def test_every_request_gets_the_tokens_it_would_get_alone():
    rng = np.random.default_rng(5)
    jobs = [(list(rng.integers(0, 5000, size=int(rng.integers(1, 9)))), int(rng.integers(1, 12))) for _ in range(11)]
    q = JobQueue(FakeExecutor(max_batch=4))
    ids = [q.submit(p, n) for p, n in jobs[:6]]
    for _ in range(5):                                       # the rest arrive while the first are being served
        q.step()
    ids += [q.submit(p, n) for p, n in jobs[6:]]
    got = q.run()
    assert sorted(got) == sorted(ids)
    for jid, (p, n) in zip(ids, jobs):
        assert got[jid] == alone(p, n)
    assert max(q.batch_sizes) == 4 and min(q.batch_sizes) >= 1
    assert not q.active and not q.waiting and len(q.free_slots) == 4


def test_requests_join_and_leave_between_steps_and_slots_are_reused():
    ex = FakeExecutor(max_batch=2)
    q = JobQueue(ex)
    a = q.submit([1, 2, 3], 2)          # 3 prompt steps (the third gives token 1) + 1 more step
    b = q.submit([4], 1)                # one step
    c = q.submit([5, 6], 3)             # waits for a slot
    assert q.step() == 2                # a, b
    assert q.finished[b].output == alone([4], 1) and q.finished[b].left_at_step == 1
    assert q.step() == 2                # a, c: c took b's slot at once
    assert q.active[1].slot == q.finished[b].slot and q.active[1].joined_at_step == 1
    q.run()
    assert q.finished[a].output == alone([1, 2, 3], 2)
    assert q.finished[c].output == alone([5, 6], 3)
    # positions of a request are consecutive from 0 in its slot
    seen = {}
    for tokens, slots, positions in ex.calls:
        for s, p in zip(slots, positions):
            if p == 0:
                seen[s] = 0
            else:
                assert p == seen[s] + 1
                seen[s] = p
    assert q.steps == len(ex.calls)     # one micro-batch per step, never two in flight


def test_end_of_sequence_token_and_argument_checks():
    prompt = [9, 9, 9]
    full = alone(prompt, 6)
    q = JobQueue(FakeExecutor(max_batch=3))
    j = q.submit(prompt, 6, eos_token=full[2])
    assert q.run()[j] == full[:3]
    with pytest.raises(ValueError):
        q.submit([], 3)
    with pytest.raises(ValueError):
        q.submit([1], 0)
    with pytest.raises(ValueError):
        q.submit([1] * 60, 10)              # 69 positions in a cache of 64
    with pytest.raises(ValueError):
        JobQueue(FakeExecutor(max_batch=2), max_batch=3)
    assert JobQueue(FakeExecutor()).step() == 0
