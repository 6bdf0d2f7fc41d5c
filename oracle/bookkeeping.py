"""Integer model of the paged KV pool.  Test infrastructure only (see oracle/__init__).

What the paper fixes (Section 2.3 "Decoding"): a forked sequence shares its parent's
prefix; on a paged cache the fork maps the parent's blocks into the child and physically
duplicates no more than a single block; a finished sequence gives back exactly the cache
that no other sequence still holds.

What the paper leaves open and this model decides (the CUDA library documents the same
policy in its header so that block ids can be compared one by one):
  * the child receives the private copy of the partial last block, at fork time; the
    parent keeps its own block and goes on appending in place;
  * the free list is a stack: a fresh pool hands out 0, 1, 2, ...; released blocks are
    pushed in table order and reused last-in first-out;
  * thread ids come from a counter and are never reused;
  * a batched call is processed in index order and changes nothing if any entry fails.
"""
from __future__ import annotations


class BookkeepingError(Exception):
    def __init__(self, code: str):
        super().__init__(code)
        self.code = code


class BlockModel:
    def __init__(self, num_blocks: int, block_size: int, max_threads: int,
                 max_blocks_per_thread: int):
        self.num_blocks = num_blocks
        self.block_size = block_size
        self.max_threads = max_threads
        self.max_blocks_per_thread = max_blocks_per_thread
        self.free = list(range(num_blocks - 1, -1, -1))   # pop() yields 0, 1, 2, ...
        self.refcount = [0] * num_blocks
        self.tables = {}      # live thread id -> list of block ids
        self.lens = {}        # live thread id -> tokens
        self.next_tid = 0
        self.cow_blocks = 0   # blocks copied by forks so far
        self.cow_rows = 0     # token rows copied by forks so far
        self.peak_used = 0    # most blocks in use at once so far

    # ------------------------------------------------------------ helpers
    def _alloc(self) -> int:
        b = self.free.pop()
        assert self.refcount[b] == 0
        self.refcount[b] = 1
        self.peak_used = max(self.peak_used, self.num_blocks - len(self.free))
        return b

    def _check_live(self, tids):
        for t in tids:
            if t not in self.tables:
                raise BookkeepingError("BAD_THREAD")

    # ------------------------------------------------------------ operations
    def new_threads(self, n: int):
        if len(self.tables) + n > self.max_threads:
            raise BookkeepingError("NO_THREADS")
        out = []
        for _ in range(n):
            t = self.next_tid
            self.next_tid += 1
            self.tables[t] = []
            self.lens[t] = 0
            out.append(t)
        return out

    def fork(self, parents):
        """Returns (children, copies); copies = [(src_block, dst_block, rows)] in order."""
        self._check_live(parents)
        if len(self.tables) + len(parents) > self.max_threads:
            raise BookkeepingError("NO_THREADS")
        B = self.block_size
        need = sum(1 for p in parents if self.lens[p] % B != 0)
        if need > len(self.free):
            raise BookkeepingError("NO_BLOCKS")
        children, copies = [], []
        for p in parents:
            L = self.lens[p]
            full, r = divmod(L, B)
            table = list(self.tables[p][:full])          # shared: same block ids
            for b in table:
                self.refcount[b] += 1
            if r:                                        # at most one block is copied
                dst = self._alloc()
                copies.append((self.tables[p][full], dst, r))
                table.append(dst)
                self.cow_blocks += 1
                self.cow_rows += r
            c = self.next_tid
            self.next_tid += 1
            self.tables[c] = table
            self.lens[c] = L
            children.append(c)
        return children, copies

    def append(self, tids, n_tok=None):
        """Returns, per thread, the list of (block, offset) slots its new rows go to."""
        n_tok = [1] * len(tids) if n_tok is None else list(n_tok)
        self._check_live(tids)
        if len(set(tids)) != len(tids) or any(n < 0 for n in n_tok):
            raise BookkeepingError("INVALID_ARG")
        B = self.block_size
        need = 0
        for t, n in zip(tids, n_tok):
            blocks_after = -(-(self.lens[t] + n) // B)
            if blocks_after > self.max_blocks_per_thread:
                raise BookkeepingError("TABLE_FULL")
            need += blocks_after - len(self.tables[t])
        if need > len(self.free):
            raise BookkeepingError("NO_BLOCKS")
        slots = []
        for t, n in zip(tids, n_tok):
            mine = []
            for _ in range(n):
                pos = self.lens[t]
                if pos % B == 0:
                    self.tables[t].append(self._alloc())
                mine.append((self.tables[t][pos // B], pos % B))
                self.lens[t] = pos + 1
            slots.append(mine)
        return slots

    def release(self, tids):
        """ReleaseCache: drop one reference per table entry; free what reaches zero."""
        self._check_live(tids)
        if len(set(tids)) != len(tids):
            raise BookkeepingError("BAD_THREAD")
        for t in tids:
            for b in self.tables[t]:
                self.refcount[b] -= 1
                if self.refcount[b] == 0:
                    self.free.append(b)
            del self.tables[t]
            del self.lens[t]

    def accept(self, tids, n_cand, n_keep):
        """Outcome of a predict-verify step (Section 3.2 "Implementation", the Medusa setting):
        the last n_cand rows of a thread are speculated tokens, n_keep of them are kept (the
        accepted ones, moved up behind the committed rows) and the rest is dropped.  Blocks
        that hold no remaining row go back to the pool, in table order.  The blocks from the
        first candidate on must belong to this thread alone (nobody forked from it meanwhile).
        Returns nothing: which rows are kept does not matter to the tables."""
        self._check_live(tids)
        if len(set(tids)) != len(tids):
            raise BookkeepingError("INVALID_ARG")
        B = self.block_size
        for t, k, keep in zip(tids, n_cand, n_keep):
            if not (1 <= k <= 64 and k <= self.lens[t] and 0 <= keep <= k):
                raise BookkeepingError("INVALID_ARG")
            first = (self.lens[t] - k) // B
            if any(self.refcount[b] != 1 for b in self.tables[t][first:]):
                raise BookkeepingError("INVALID_ARG")
        for t, k, keep in zip(tids, n_cand, n_keep):
            new_len = self.lens[t] - k + keep
            blocks = -(-new_len // B)
            for b in self.tables[t][blocks:]:
                self.refcount[b] = 0
                self.free.append(b)
            del self.tables[t][blocks:]
            self.lens[t] = new_len

    # ------------------------------------------------------------ counters
    def free_list(self):
        """Block ids in the order they would be handed out next."""
        return self.free[::-1]

    def used_blocks(self) -> int:
        return sum(1 for c in self.refcount if c > 0)

    def unique_tokens(self, tids) -> int:
        """KV slots needed to hold the chains of `tids` with sharing (cached tokens)."""
        B = self.block_size
        rows = {}
        for t in tids:
            for i, b in enumerate(self.tables[t]):
                rows[b] = max(rows.get(b, 0), min(B, self.lens[t] - i * B))
        return sum(rows.values())

    def attended_tokens(self, tids) -> int:
        """Sum over threads of the tokens attended when predicting the next token."""
        return sum(self.lens[t] for t in tids)
