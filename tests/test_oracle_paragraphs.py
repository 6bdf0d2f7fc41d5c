"""Pin for the paragraph-tree checker: the worked example of the paper's decoding figure
(a response p0 - p1 - p2 whose paragraphs each have a root sentence and a detail part, Fig. 3
caption) must restore to the sequential text, with the order written out by hand."""
from oracle import CHILD, EOS, FORK, SequenceGroup


def test_three_paragraph_response_restores_in_reading_order():
    # scripted model: per sequence, the tokens it will emit
    script = {
        0: ["r0a", "r0b", FORK, "r1a", FORK, "r2a", "r2b", EOS],   # roots of p0, p1, p2
        1: ["d0a", "d0b", "d0c", EOS],                              # detail of p0
        2: ["d1a", EOS],                                            # detail of p1
    }
    g = SequenceGroup(["P0", "P1"])
    pos = {}

    def sample(s):
        i = g.seqs.index(s)
        pos[i] = pos.get(i, 0) + 1
        return script[i][pos[i] - 1]

    while not all(s.finished for s in g.seqs):
        g.step(sample)
    # by hand: root part of p0 (incl. its fork token), detail of p0 (thread 1, after the forced
    # child token), root of p1, detail of p1 (thread 2), rest of thread 0
    assert g.restore() == ["r0a", "r0b", FORK, "d0a", "d0b", "d0c", EOS,
                           "r1a", FORK, "d1a", EOS, "r2a", "r2b", EOS]
    assert g.seqs[1].tokens[:6] == ["P0", "P1", "r0a", "r0b", FORK, CHILD]
    assert g.slices() == [(0, 2, 5), (1, 6, 10), (0, 5, 7), (2, 8, 10), (0, 7, 10)]


def test_a_detail_thread_that_forks_again_is_read_depth_first():
    # Worked by hand from Algorithm 1's traversal (root, first child, next sibling): the detail
    # thread of the first paragraph forks itself, so its own detail comes before its remainder,
    # and both come before the remainder of the root thread.
    script = {0: ["a", FORK, "b", EOS], 1: ["c", FORK, "d", EOS], 2: ["e", EOS]}
    g = SequenceGroup(["P"])
    pos = {}

    def sample(s):
        i = g.seqs.index(s)
        pos[i] = pos.get(i, 0) + 1
        return script[i][pos[i] - 1]

    passes = 0
    while not all(s.finished for s in g.seqs):
        g.step(sample)
        passes += 1
    assert passes == 8                      # a thread born in a pass first decodes in the next
    assert g.seqs[0].tokens == ["P", "a", FORK, "b", EOS]
    assert g.seqs[1].tokens == ["P", "a", FORK, CHILD, "c", FORK, "d", EOS]
    assert g.seqs[2].tokens == ["P", "a", FORK, CHILD, "c", FORK, CHILD, "e", EOS]
    assert g.slices() == [(0, 1, 3), (1, 4, 6), (2, 7, 9), (1, 6, 8), (0, 3, 5)]
    assert g.restore() == ["a", FORK, "c", FORK, "e", EOS, "d", EOS, "b", EOS]
