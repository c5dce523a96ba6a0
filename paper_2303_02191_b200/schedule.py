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


def chains(ops, rounds, reads, write, is_conv, max_items=20, min_width=2):
    """Issue order of a program whose dependent convolutions may share launches (rtoss_conv_chain).

    Walks the rounds of `levels` in order and collects the convolutions (is_conv(op)) of consecutive rounds into
    segments of at most max_items; an operation of another kind ends the segment before it is issued (it may read what
    the segment writes), and so do a round that would not fit and a round of fewer than min_width convolutions (which
    is issued on its own).  Returns a list of steps:
      ('chain', [op indices in issue order], [after masks])  -- bit j of after[i]: item i reads what item j (earlier
                                                                 in the same segment) writes
      ('op', op index)                                        -- issued on its own
    Every buffer region is written once per pass, so reads-after-writes are the only dependencies inside a segment."""
    steps, seg = [], []

    def flush():
        if len(seg) == 1:
            steps.append(("op", seg[0]))
        elif seg:
            pos = {i: q for q, i in enumerate(seg)}
            writer = {}
            for i in seg:
                writer.setdefault(write(ops[i]), []).append(i)
            after = []
            for i in seg:
                m = 0
                for r in reads(ops[i]):
                    for j in writer.get(r, ()):
                        if pos[j] < pos[i]:
                            m |= 1 << pos[j]
                after.append(m)
            steps.append(("chain", list(seg), after))
        del seg[:]

    for rnd in rounds:
        convs = [i for i in rnd if is_conv(ops[i])]
        rest = [i for i in rnd if not is_conv(ops[i])]
        if len(convs) < min_width:
            # a round of one convolution gains nothing inside a shared launch (the wait inside the kernel costs about a
            # microsecond more than the boundary between two launches): it ends the segment and goes out alone
            flush()
            steps.extend(("op", i) for i in convs + rest)
            continue
        if len(seg) + len(convs) > max_items:
            flush()
        while len(convs) > max_items:     # a round wider than a launch
            seg.extend(convs[:max_items])
            convs = convs[max_items:]
            flush()
        seg.extend(convs)
        if rest:
            flush()
            steps.extend(("op", i) for i in rest)
    flush()
    return steps
