"""CPU oracle for the integer side of continuous depth batching: which (sequence, token, loop
depth) items share each recurrent pass, and which KV pages a sequence owns.

TEST INFRASTRUCTURE (see cdb_oracle.py).  Works on exit-depth traces only, no tensors.

Follows section 4.1 and Fig. 1 of the paper: a fixed number of batch slots; a token occupies a
slot for r_t consecutive recurrent passes; boundary stages (coda, sampling, prelude) take no
recurrent pass.
  * refill: a slot freed by an exit is taken in the very next pass by the next token of the same
    sequence, or, when that sequence is finished, by the first token of the next waiting sequence;
  * no-refill: all live sequences start a token together, exited tokens leave their slot idle
    until the slowest token of the round has exited; only then does the next round start.
"""
from __future__ import annotations


def simulate(traces, slots, mode="refill"):
    """traces[s] = exit depths of the tokens of sequence s, in order.  Sequences are admitted in
    index order, lowest free slot first.  Returns grid[pass][slot] = (seq, token index, depth)
    or None for an idle slot."""
    waiting = list(range(len(traces)))
    owner = [None] * slots                       # slot -> [seq, token index, depth] or None
    grid = []

    def admit(slot):
        while waiting:
            s = waiting.pop(0)
            if traces[s]:
                owner[slot] = [s, 0, 0]
                return
        owner[slot] = None

    for k in range(slots):
        admit(k)
    while any(o is not None for o in owner):
        if mode == "refill":
            row = []
            for k in range(slots):
                o = owner[k]
                if o is None:
                    row.append(None)
                    continue
                o[2] += 1
                row.append(tuple(o))
            grid.append(row)
            for k in range(slots):
                o = owner[k]
                if o is not None and o[2] == traces[o[0]][o[1]]:        # token exits after this pass
                    if o[1] + 1 < len(traces[o[0]]):
                        owner[k] = [o[0], o[1] + 1, 0]
                    else:
                        admit(k)
        elif mode == "no_refill":
            depth = max(traces[o[0]][o[1]] for o in owner if o is not None)
            for r in range(1, depth + 1):
                grid.append([tuple([o[0], o[1], r]) if o is not None and r <= traces[o[0]][o[1]] else None
                             for o in owner])
            for k in range(slots):
                o = owner[k]
                if o is None:
                    continue
                if o[1] + 1 < len(traces[o[0]]):
                    owner[k] = [o[0], o[1] + 1, 0]
                else:
                    admit(k)
        else:
            raise ValueError(mode)
    return grid


def recurrent_passes(traces, slots, mode):
    return len(simulate(traces, slots, mode))


def refill_lower_bound(traces, slots):
    total = sum(sum(t) for t in traces)
    return -(-total // slots)


class PageAllocator:
    """16-token pages handed out from a stack that first yields 0, 1, 2, ...; a finished sequence
    returns its pages so that they are handed out again in the same logical order.  A sequence
    takes a new page when its next position is a multiple of the page size."""

    def __init__(self, n_pages, page_size=16):
        self.page_size = page_size
        self.free = list(range(n_pages - 1, -1, -1))        # pop() -> lowest id first
        self.table = {}                                     # seq -> list of physical pages

    def ensure(self, seq, position):
        """Make sure `position` of `seq` is backed by a page; returns the sequence's table."""
        pages = self.table.setdefault(seq, [])
        while len(pages) * self.page_size <= position:
            if not self.free:
                raise MemoryError("page pool exhausted")
            pages.append(self.free.pop())
        return pages

    def release(self, seq):
        for p in reversed(self.table.pop(seq, [])):
            self.free.append(p)
