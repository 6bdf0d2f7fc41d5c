"""Paragraph tree of Algorithm 1 on plain token lists.  Test infrastructure only.

Follows the algorithm's own bookkeeping: a sequence group holds the sequences of one prompt;
every sequence tracks the leaf paragraph node at its end; when a sequence whose last token is
the fork token is duplicated, the current node is closed, a next-sibling node (same sequence)
and a first-child node (the copy, after its forced child token) are opened; Restore walks the
tree root, first child, next sibling and concatenates the slices.
"""
from __future__ import annotations

FORK, CHILD, EOS = "[Fork]", "[Child]", "[EOS]"


class PNode:
    def __init__(self, seq, start):
        self.seq, self.start, self.end = seq, start, None
        self.first_child = None
        self.next_sibling = None


class Sequence:
    def __init__(self, tokens):
        self.tokens = list(tokens)
        self.finished = False
        self.current_node = None


class SequenceGroup:
    def __init__(self, prompt_tokens):
        p = Sequence(prompt_tokens)
        self.root = PNode(p, len(p.tokens))
        p.current_node = self.root
        self.seqs = [p]

    def step(self, sample):
        """One AparDecode pass.  sample(seq) returns the next token of an unfinished sequence."""
        for s in list(self.seqs):
            if s.finished:
                continue
            x = sample(s)
            if s.tokens[-1] == FORK:
                c = Sequence(s.tokens)
                c.tokens.append(CHILD)
                self.seqs.append(c)
                n, nc = PNode(s, len(s.tokens)), PNode(c, len(c.tokens))
                s.current_node.end = len(s.tokens)
                s.current_node.next_sibling = n
                s.current_node.first_child = nc
                s.current_node = n
                c.current_node = nc
            s.tokens.append(x)
            if x == EOS:
                s.finished = True

    def slices(self):
        """(sequence index, start, end) in Restore order; an open end is the sequence's length."""
        out = []

        def visit(n):
            out.append((self.seqs.index(n.seq), n.start,
                        len(n.seq.tokens) if n.end is None else n.end))
            if n.first_child is not None:
                visit(n.first_child)
            if n.next_sibling is not None:
                visit(n.next_sibling)
        visit(self.root)
        return out

    def restore(self):
        return [t for i, a, b in self.slices() for t in self.seqs[i].tokens[a:b]]
