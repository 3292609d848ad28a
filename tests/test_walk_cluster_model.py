"""A host-side model of how the blocks of the sampling walk's cluster share p between passes.

Every block of the cluster follows the whole walk; after a rejection each block rewrites its own
share of the residual distribution p and all blocks meet at one cluster barrier.  The decision
for the next child then reads one entry of p, which may lie in another block's share.  Nothing
but that barrier orders the blocks, so a block that is already in the next pass must not be able
to overwrite the entry a slower block has yet to read: p exists twice and a pass writes the
copy it does not read.  The model runs the blocks as coroutines under many random schedules and
checks that every decision read returns the value of the pass it belongs to; with a single copy
the same schedules produce stale reads, which is the mistake the second copy is there for.
No GPU is involved: on the device such a race would only show as a rare wrong token."""
import random

N_BLOCKS = 8
SHARE = 4                      # entries of p per block


class Cluster:
    def __init__(self, copies):
        self.copies = copies
        # p[copy][entry] = number of the pass that wrote it (0 = the lazy distribution)
        self.p = [[0] * (N_BLOCKS * SHARE) for _ in range(copies)]
        self.arrived = 0
        self.generation = 0
        self.stale = []          # (block, pass, value read)


def block(cl, rank, n_passes, tokens):
    cur = 0                      # which copy holds the current p
    for k in range(1, n_passes + 1):
        # decision of pass k's child: one entry of the current p, anywhere in the vocabulary
        got = cl.p[cur % cl.copies][tokens[k - 1]]
        if got != k - 1:
            cl.stale.append((rank, k, got))
        yield
        # rejection: this block's share of the new p goes to the copy it does not read
        nxt = (cur + 1) % cl.copies
        for v in range(rank * SHARE, (rank + 1) * SHARE):
            cl.p[nxt][v] = k
            yield
        cur = nxt
        # cluster barrier (arrive, then wait for the generation to move on)
        gen = cl.generation
        cl.arrived += 1
        if cl.arrived == N_BLOCKS:
            cl.arrived = 0
            cl.generation += 1
        while cl.generation == gen:
            yield


def run(copies, seed, n_passes=6):
    rng = random.Random(seed)
    cl = Cluster(copies)
    tokens = [rng.randrange(N_BLOCKS * SHARE) for _ in range(n_passes)]
    live = [block(cl, r, n_passes, tokens) for r in range(N_BLOCKS)]
    ticks = 0
    while live:
        ticks += 1
        assert ticks < 200000, "the model itself hung"
        g = rng.choice(live)     # any interleaving the hardware could produce
        try:
            next(g)
        except StopIteration:
            live.remove(g)
    return cl


def test_two_copies_never_give_a_decision_a_value_of_another_pass():
    for seed in range(300):
        cl = run(2, seed)
        assert cl.stale == [], (seed, cl.stale[:3])


def test_one_copy_lets_a_faster_block_overwrite_what_a_slower_one_still_reads():
    bad = sum(1 for seed in range(300) if run(1, seed).stale)
    assert bad > 0
    # and what is read then is always the NEXT pass's value: the overwrite, nothing else
    for seed in range(300):
        for _, k, got in run(1, seed).stale:
            assert got == k
