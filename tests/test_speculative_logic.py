"""Accept/reject logic of the speculative loop with toy models (no GPU): the output must be the target's own
greedy sequence whatever the draft proposes, and both caches must only ever be read where they are valid."""
import numpy as np
import pytest

from paper_2504_08791_b200.speculative import SpeculativeDecoder


class ToyModel:
    """A 'model' whose next token depends on the whole history; keeps a cache like the real contexts do and
    fails if a step reads a position that was never written or was written with a token that is not the
    sequence's token there (as a stale cache entry would be)."""

    def __init__(self, vocab, salt, prefix):
        self.vocab, self.salt = vocab, salt
        self.cache = list(prefix)            # token consumed at each position
        self.steps = 0

    def _next(self, hist):
        h = self.salt
        for i, t in enumerate(hist):
            h = (h * 1000003 + (t + 1) * (i + 7)) % 2147483647
        return h % self.vocab

    def step(self, tokens, pos):
        assert 1 <= len(tokens) <= 8
        assert pos <= len(self.cache), "a step may not leave a hole in the cache"
        self.steps += 1
        out = []
        for i, t in enumerate(tokens):
            p = pos + i
            if p < len(self.cache):
                self.cache[p] = t
                del self.cache[p + 1:]       # later entries are stale from now on
            else:
                self.cache.append(t)
            out.append(self._next(self.cache[:p + 1]))
        return np.array(out, np.int32)


def greedy(model_salt, vocab, prefix, first, n):
    m = ToyModel(vocab, model_salt, prefix)
    toks, tok, pos = [], first, len(prefix)
    for _ in range(n):
        tok = int(m.step([tok], pos)[0])
        pos += 1
        toks.append(tok)
    return toks


class MixedDraft(ToyModel):
    """Agrees with the target except at the steps listed in `wrong`."""

    def __init__(self, vocab, salt, prefix, wrong):
        super().__init__(vocab, salt, prefix)
        self.wrong, self.calls = set(wrong), 0

    def step(self, tokens, pos):
        out = super().step(tokens, pos)
        self.calls += 1
        if self.calls in self.wrong:
            out = (out + 1) % self.vocab
        return out


@pytest.mark.parametrize("n_draft", [1, 3, 4, 7])
@pytest.mark.parametrize("kind", ["perfect", "unrelated", "mixed"])
def test_output_equals_plain_greedy_decoding(n_draft, kind):
    vocab, prefix, first, n = 50, [3, 1, 4, 1, 5, 9, 2, 6], 7, 41
    want = greedy(11, vocab, prefix, first, n)
    target = ToyModel(vocab, 11, prefix)
    if kind == "perfect":
        draft = ToyModel(vocab, 11, prefix)
    elif kind == "unrelated":
        draft = ToyModel(vocab, 12, prefix)
    else:
        draft = MixedDraft(vocab, 11, prefix, wrong=range(2, 200, 3))
    dec = SpeculativeDecoder.from_steppers(target, draft, n_draft=n_draft, capacity=10_000)
    got, stats = dec.generate(first, len(prefix), n)
    assert got == want
    assert all(1 <= c <= n_draft + 1 for c in stats.per_cycle)
    assert stats.cycles == target.steps
    if kind == "perfect":
        assert stats.accepted == stats.proposed and stats.cycles == -(-n // (n_draft + 1))
    if kind == "unrelated":
        assert stats.cycles >= n // 2          # a draft that shares nothing is confirmed only by chance
    if kind == "mixed":
        assert 0 < stats.accepted < stats.proposed


def test_capacity_and_argument_checks():
    vocab, prefix = 20, [1, 2, 3]
    t, d = ToyModel(vocab, 1, prefix), ToyModel(vocab, 1, prefix)
    with pytest.raises(ValueError):
        SpeculativeDecoder.from_steppers(t, d, n_draft=8, capacity=100)
    dec = SpeculativeDecoder.from_steppers(t, d, n_draft=4, capacity=6)      # room for positions 3, 4, 5 only
    with pytest.raises(ValueError):
        dec.generate(0, len(prefix), 10)
