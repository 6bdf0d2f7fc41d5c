"""Restoring the sequential text of an APAR generation from its fork history, on plain token
lists.  Test infrastructure only (see oracle/__init__).

Algorithm 1 keeps a paragraph tree beside the sequences and reads the answer off it in the
order root, first child, next sibling.  What that traversal produces has a direct description,
which is what this file implements (no tree, no node objects): the text of a sequence, read
from some start position, is

    its own tokens up to the position where it first forked after that start,
    then the whole text of the sequence born there (read from just after the forced child
    token that opened it),
    then the text of the same sequence read from the fork position on.

So it is enough to remember, per sequence, at which of its positions a copy was made and which
sequence the copy became.  The hand-worked example of tests/test_oracle_paragraphs.py pins the
result; the behaviour checked is Algorithm 1's (decode pass, fork rule, Restore order).
"""
from __future__ import annotations

FORK, CHILD, EOS = "[Fork]", "[Child]", "[EOS]"


class Thread:
    """One generation thread: its tokens and the copies made of it, as (position, index of the
    new thread in the group), in the order they were made (positions increase)."""

    def __init__(self, tokens):
        self.tokens = list(tokens)
        self.finished = False
        self.births = []


class SequenceGroup:
    """All threads generated for one prompt (Section 2.3 "Sequence and sequence group")."""

    def __init__(self, prompt_tokens):
        self.seqs = [Thread(prompt_tokens)]
        self.answer_from = len(self.seqs[0].tokens)     # the prompt is not part of the answer

    def step(self, sample):
        """One decode pass over the threads that exist when it begins.  `sample(thread)` gives
        the next token of an unfinished thread.  A thread whose newest token is the fork token
        is copied before its new token is added; the copy starts with the forced child token
        and first decodes in the next pass."""
        for k in range(len(self.seqs)):
            th = self.seqs[k]
            if th.finished:
                continue
            token = sample(th)
            if th.tokens[-1] == FORK:
                th.births.append((len(th.tokens), len(self.seqs)))
                self.seqs.append(Thread(th.tokens + [CHILD]))
            th.tokens.append(token)
            th.finished = token == EOS

    def slices(self):
        """(thread index, start, end) pieces whose concatenation is the answer."""
        pieces = []

        def read(k, start):
            th = self.seqs[k]
            for at, born in th.births:
                pieces.append((k, start, at))
                read(born, at + 1)          # skip the child token the copy was opened with
                start = at
            pieces.append((k, start, len(th.tokens)))

        read(0, self.answer_from)
        return pieces

    def restore(self):
        return [tok for k, a, b in self.slices() for tok in self.seqs[k].tokens[a:b]]
