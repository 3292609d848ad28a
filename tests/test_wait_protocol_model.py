"""A host-side model of the bounded-wait protocol the tensor-core kernels use (producer -> MMA
issuer -> epilogue warps, handing stages, accumulators and work items over through phase barriers).

On the GPU a wait that never ends would hang a device that other people share, so no test makes
one expire there.  What can be checked without a GPU is the protocol itself: every wait has a
budget; the role whose wait runs out records JK_ERR_TIMEOUT once, raises the CTA's abort flag and
returns; every other role notices the flag at its next wait and returns too; the common exit path
(drain the copies in flight, free the tensor memory) is reached by all of them.  The model below
follows the roles of the streaming GEMM: the producer takes work items from a counter, announces
each to the epilogue warps through a four-entry queue, tags every stage with "first / last k step
of its item" and closes with an end-of-work stage; the MMA issuer follows the tags; four epilogue
warps drain the two accumulators.  Same barriers, arrival counts and parities as the kernel; the
failure is injected on the host by under-filling one arrival count."""
import itertools

JK_ERR_TIMEOUT = -8
BUDGET = 200                     # scheduler ticks a wait may spin
ITEM_Q = 4
FIRST, LAST, END = 1, 2, 4


class PhaseBarrier:
    """mbarrier: `count` arrivals complete a phase; waiters test the parity of the phase."""

    def __init__(self, count):
        self.count, self.pending, self.phase = count, count, 0

    def arrive(self):
        self.pending -= 1
        if self.pending == 0:
            self.pending = self.count
            self.phase ^= 1

    def done(self, parity):      # try_wait.parity: true once the phase with that parity is over
        return self.phase != parity


class Cta:
    def __init__(self, stages, epilogue_warps=4):
        self.full = [PhaseBarrier(1) for _ in range(stages)]
        self.empty = [PhaseBarrier(1) for _ in range(stages)]
        self.acc_full = [PhaseBarrier(1) for _ in range(2)]
        self.acc_empty = [PhaseBarrier(epilogue_warps) for _ in range(2)]
        self.iq_full = [PhaseBarrier(1) for _ in range(ITEM_Q)]
        self.iq_empty = [PhaseBarrier(epilogue_warps) for _ in range(ITEM_Q)]
        self.st_flag = [0] * stages
        self.q_item = [0] * ITEM_Q
        self.abort = False
        self.status = 0
        self.timeouts = 0
        self.exited = []
        self.tmem_freed = False
        self.stored = []             # (warp, item) pairs the epilogue warps wrote


def bounded_wait(cta, bar, parity):
    """Generator: yields while spinning; returns False on expiry or when another role gave up."""
    for _ in range(BUDGET):
        if bar.done(parity):
            return True
        if cta.abort:
            return False
        yield
    cta.abort = True
    cta.timeouts += 1
    if cta.status == 0:          # compare-and-swap on 0: the first error stays
        cta.status = JK_ERR_TIMEOUT
    return False


def producer(cta, counter, total_items, units_of, stages):
    s, ph, issued, qn = 0, 0, 0, 0
    ok = True
    while ok:
        item = counter[0]
        counter[0] += 1                                  # atomicAdd on the global counter
        if item >= total_items:
            break
        qs = qn % ITEM_Q
        if qn >= ITEM_Q:
            ok = yield from bounded_wait(cta, cta.iq_empty[qs], ((qn // ITEM_Q) - 1) & 1)
            if not ok:
                break
        cta.q_item[qs] = item
        cta.iq_full[qs].arrive()
        qn += 1
        n = units_of(item)
        for k in range(n):
            if issued >= stages:
                ok = yield from bounded_wait(cta, cta.empty[s], ph ^ 1)
                if not ok:
                    break
            cta.st_flag[s] = (FIRST if k == 0 else 0) | (LAST if k == n - 1 else 0)
            cta.full[s].arrive()                         # the copies land: expect_tx completes
            issued += 1
            s += 1
            if s == stages:
                s, ph = 0, ph ^ 1
            yield
    if ok:
        qs = qn % ITEM_Q
        if qn >= ITEM_Q:
            ok = yield from bounded_wait(cta, cta.iq_empty[qs], ((qn // ITEM_Q) - 1) & 1)
        if ok:
            cta.q_item[qs] = -1
            cta.iq_full[qs].arrive()
            if issued >= stages:
                ok = yield from bounded_wait(cta, cta.empty[s], ph ^ 1)
        if ok:
            cta.st_flag[s] = END
            cta.full[s].arrive()
    cta.exited.append("producer")


def mma(cta, stages):
    s, fph, seg, acc = 0, 0, 0, 0
    while True:
        ok = yield from bounded_wait(cta, cta.full[s], fph)
        if not ok:
            break
        flag = cta.st_flag[s]
        if flag & END:
            break
        if flag & FIRST:
            acc = seg & 1
            if seg >= 2:
                ok = yield from bounded_wait(cta, cta.acc_empty[acc], ((seg >> 1) & 1) ^ 1)
                if not ok:
                    break
        cta.empty[s].arrive()                            # tcgen05.commit -> the stage is free
        if flag & LAST:
            cta.acc_full[acc].arrive()
            seg += 1
        s += 1
        if s == stages:
            s, fph = 0, fph ^ 1
        yield
    cta.exited.append("mma")


def epilogue(cta, warp, arrives=True):
    seg, qn = 0, 0
    while True:
        qs = qn % ITEM_Q
        ok = yield from bounded_wait(cta, cta.iq_full[qs], (qn // ITEM_Q) & 1)
        if not ok:
            break
        item = cta.q_item[qs]
        cta.iq_empty[qs].arrive()
        qn += 1
        if item < 0:
            break
        acc = seg & 1
        ok = yield from bounded_wait(cta, cta.acc_full[acc], (seg >> 1) & 1)
        if not ok:
            break
        yield                                            # drain the accumulator to slot `item`
        cta.stored.append((warp, item))
        if arrives:
            cta.acc_empty[acc].arrive()
        seg += 1
    cta.exited.append(f"epilogue{warp}")


def run(n_ctas=3, total_items=17, stages=3, silent_warp=None, max_ticks=100000):
    """Several CTAs share one item counter; the failing CTA (if any) is the first."""
    counter = [0]
    units_of = lambda item: 1 + item % 4                 # chunks of different lengths
    ctas = [Cta(stages) for _ in range(n_ctas)]
    live = []
    for i, cta in enumerate(ctas):
        roles = [producer(cta, counter, total_items, units_of, stages), mma(cta, stages)]
        roles += [epilogue(cta, w, arrives=not (i == 0 and w == silent_warp)) for w in range(4)]
        live += roles
    for tick in itertools.count():
        assert tick < max_ticks, "the model itself hung: a wait without a budget"
        if not live:
            break
        for r in list(live):
            try:
                next(r)
            except StopIteration:
                live.remove(r)
    for cta in ctas:
        cta.tmem_freed = True                            # the exit path behind __syncthreads()
    return ctas, tick


ROLES = sorted(["producer", "mma"] + [f"epilogue{w}" for w in range(4)])


def test_all_roles_finish_and_every_item_is_stored_once_per_warp():
    ctas, _ = run()
    for cta in ctas:
        assert cta.status == 0 and not cta.abort and cta.timeouts == 0
        assert sorted(cta.exited) == ROLES and cta.tmem_freed
    # every item went to exactly one CTA, and all four epilogue warps of that CTA stored it
    owner = {}
    for i, cta in enumerate(ctas):
        for warp, item in cta.stored:
            owner.setdefault(item, set()).add(i)
        for item in {it for _, it in cta.stored}:
            assert sorted(w for w, it in cta.stored if it == item) == [0, 1, 2, 3]
    assert sorted(owner) == list(range(17)) and all(len(v) == 1 for v in owner.values())


def test_an_underfilled_arrival_count_expires_one_wait_and_unwinds_every_role():
    # epilogue warp 2 of the first CTA never releases the accumulators: 3 of 4 arrivals
    ctas, ticks = run(silent_warp=2)
    bad = ctas[0]
    assert bad.status == JK_ERR_TIMEOUT and bad.abort
    # the roles that were already waiting when the arrival went missing run out together, the
    # rest see the flag; the status word keeps one error whatever the number
    assert 1 <= bad.timeouts <= 6
    assert sorted(bad.exited) == ROLES and bad.tmem_freed
    for cta in ctas[1:]:                             # the other CTAs wait for nobody and finish
        assert cta.status == 0 and sorted(cta.exited) == ROLES
    assert ticks < 20 * BUDGET                       # bounded: no role outlived the budget by much


def test_the_first_error_is_kept():
    cta2 = Cta(2)
    cta2.status = -9                                 # an earlier bounds error
    g = bounded_wait(cta2, PhaseBarrier(1), 0)
    for _ in g:
        pass
    assert cta2.status == -9 and cta2.abort
