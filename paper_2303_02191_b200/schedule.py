"""Launch schedule of a chained network program: which operations may run side by side.

A program is a list of operations, each reading some buffers and writing one (possibly a channel slice of it).
Every buffer region is written once per pass, so the only dependencies are producer -> consumer.  `levels` sorts
the operations into rounds such that an operation's round is later than the rounds of the producers of what it
reads.  Operations of one round do not depend on one another; the network runners hand the convolutions of a round
to rtoss_conv_group (one launch for those that can share it) and run the rest one by one.
"""


def levels(ops, reads, write, late=True):
    """ops: list; reads(op) -> iterable of buffer names; write(op) -> buffer name (or None).
    Returns a list of rounds, each a list of op indices in program order.  late: every operation sits in the LAST
    round that still lets its consumers run when they must (as-late-as-possible; the number of rounds is that of the
    as-soon-as-possible order).  Chains of different length that end together -- the towers on a short and on a long
    branch of a pyramid -- then run layer i of every chain in one round."""
    writers = {}
    for i, op in enumerate(ops):
        w = write(op)
        if w is not None:
            writers.setdefault(w, []).append(i)
    level = [0] * len(ops)
    consumers = [[] for _ in ops]
    for i, op in enumerate(ops):
        lv = 0
        for r in reads(op):
            for j in writers.get(r, ()):
                if j >= i:
                    raise ValueError("operation %d reads %r before operation %d has written it" % (i, r, j))
                lv = max(lv, level[j] + 1)
                consumers[j].append(i)
        level[i] = lv
    if not ops:
        return []
    last = max(level)
    if late:
        for i in range(len(ops) - 1, -1, -1):
            level[i] = min([level[c] - 1 for c in consumers[i]] + [last])
    rounds = [[] for _ in range(last + 1)]
    for i, lv in enumerate(level):
        rounds[lv].append(i)
    return rounds
