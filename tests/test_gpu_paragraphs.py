"""Algorithm 1 end to end without a model: a scripted sampler drives the paragraph-tree checker
(token lists) and the library (fork / append / release + paragraph tracking); the library's
restored slices must be the checker's, and reading the checker's tokens through them must give
the restored text."""
import pytest
import torch

from oracle import CHILD, EOS, FORK, SequenceGroup
from paper_2401_06761_b200 import synth

pytestmark = pytest.mark.gpu


def test_restore_matches_algorithm_1():
    from paper_2401_06761_b200 import binding as B
    from paper_2401_06761_b200.session import PagedSession
    import random
    rnd = random.Random(4)
    shape = synth.LayerShape(8, 2)
    sess = PagedSession(shape, 400, 64, 40)
    prompt = [f"P{i}" for i in range(23)]
    g = SequenceGroup(prompt)
    z = torch.zeros((64, 2, 128), dtype=torch.bfloat16, device="cuda")
    (root,) = sess.new_threads(1)
    sess.append([root], [len(prompt)], z[:23], z[:23])
    B.apar_paragraph_root(sess.ctx, root)
    tid_of = {0: root}                      # checker sequence index -> library thread
    budget = {0: 60}
    counter = [0]
    released = set()

    def sample(s):
        i = g.seqs.index(s)
        budget[i] = budget.get(i, rnd.randrange(5, 30)) - 1
        if budget[i] <= 0:
            return EOS
        counter[0] += 1
        if len(g.seqs) < 12 and s.tokens[-1] != FORK and rnd.random() < 0.12:
            return FORK
        return f"t{counter[0]}"

    for step in range(200):
        if all(s.finished for s in g.seqs):
            break
        before = len(g.seqs)
        live_before = [i for i, s in enumerate(g.seqs) if not s.finished]
        forking = [i for i in live_before if g.seqs[i].tokens[-1] == FORK]
        g.step(sample)
        # mirror the step on the library: forks (same order), forced child tokens, one token each
        if forking:
            kids = sess.fork([tid_of[i] for i in forking])
            for j, k in enumerate(kids):
                tid_of[before + j] = k
            sess.append(kids, None, z[:len(kids)], z[:len(kids)])          # the child tokens
        sess.append([tid_of[i] for i in live_before], None, z[:len(live_before)],
                    z[:len(live_before)])
        done = [i for i in live_before if g.seqs[i].finished]
        for i, sq in enumerate(g.seqs):          # same lengths on both sides
            if i not in released:
                assert sess.thread(tid_of[i])[0] == len(sq.tokens)
        if done and step % 2 == 0:           # release some finished threads early, keep others
            sess.release([tid_of[i] for i in done])
            released.update(done)
    want = [(tid_of[i], a, b) for i, a, b in g.slices()]
    got = B.apar_restore(sess.ctx, root)
    assert got == want
    inv = {t: i for i, t in tid_of.items()}
    text = [tok for t, a, b in got for tok in g.seqs[inv[t]].tokens[a:b]]
    assert text == g.restore() and CHILD not in text and len(g.seqs) > 3
    with pytest.raises(B.AparError):
        B.apar_restore(sess.ctx, tid_of[1])            # not a root
    sess.close()
