"""Verification of a small tree of speculative tokens for one thread (the shape of the paper's
speculative-decoding setting) with nothing but fork / append / attention / release: every
candidate branch is a forked thread, so a candidate token attends the thread's context and its
own ancestors among the candidates and nothing of the sibling branches; accepting a branch keeps
that thread and releases the others."""
import pytest
import torch

from helpers import OracleBackend, assert_close, assert_same_bookkeeping
from paper_2401_06761_b200 import synth

pytestmark = pytest.mark.gpu


def test_candidate_tree_as_forked_threads():
    from paper_2401_06761_b200.session import PagedSession
    shape = synth.LayerShape(8, 2)
    sess = PagedSession(shape, 64, 16, 16, poison=True)
    orc = OracleBackend(shape, 64, 16, 16)
    g = torch.Generator(device="cuda").manual_seed(77)

    def rows(n):
        kv = torch.randn((2, n, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
        return kv[0].contiguous(), kv[1].contiguous()

    def both(fn, *a):
        x, y = getattr(sess, fn)(*a), getattr(orc, fn)(*a)
        if fn in ("new_threads", "fork"):
            assert x == y
        return x

    (t,) = both("new_threads", 1)
    both("append", [t], [37], *rows(37))                 # the thread's context
    # candidates: a -> (b -> d, c): three leaves-to-root paths [a, b, d], [a, c]
    (ta,) = both("fork", [t]);       both("append", [ta], None, *rows(1))        # a
    tab, tac = both("fork", [ta, ta])
    both("append", [tab, tac], None, *rows(2))                                    # b, c
    (tabd,) = both("fork", [tab]);   both("append", [tabd], None, *rows(1))      # d
    # one query per candidate token: the thread that ends in it
    tids = [ta, tab, tac, tabd]
    q = torch.randn((4, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    out = sess.attention(tids, q)
    assert_close(out, orc.attention(tids, q, sess.sm_scale), "candidate tokens")
    assert [sess.thread(x)[0] for x in tids] == [38, 39, 39, 40]
    # accept a, c: that branch becomes the thread; everything else is released
    both("release", [t, ta, tab, tabd])
    assert_same_bookkeeping(sess, orc.model, [tac])
    both("append", [tac], None, *rows(1))
    q1 = torch.randn((1, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    assert_close(sess.attention([tac], q1), orc.attention([tac], q1, sess.sm_scale), "after accept")
    both("release", [tac])
    assert sess.stats()["free_blocks"] == 64
    sess.close()
