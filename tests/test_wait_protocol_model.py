"""A host-side model of the bounded-wait protocol the tensor-core kernels use (producer -> MMA
issuer -> epilogue warps, handing stages and accumulators over through phase barriers).

On the GPU a wait that never ends would hang a device that other people share, so no test makes
one expire there.  What can be checked without a GPU is the protocol itself: every wait has a
budget; the role whose wait runs out records JK_ERR_TIMEOUT once, raises the CTA's abort flag and
returns; every other role notices the flag at its next wait and returns too; the common exit path
(drain the copies in flight, free the tensor memory) is reached by all of them.  The model below
follows the roles of the streaming GEMM - producer, MMA issuer, four epilogue warps, the stage ring
and the two accumulators with their arrival counts and parities (the kernel's small queue of item
ids between producer and epilogue warps follows the same pattern and is left out) - and the
failure is injected on the host by under-filling one arrival count."""
import itertools

JK_ERR_TIMEOUT = -8
BUDGET = 200                     # scheduler ticks a wait may spin


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
        self.abort = False
        self.status = 0
        self.timeouts = 0
        self.exited = []
        self.tmem_freed = False


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


def producer(cta, n_units, stages):
    s, ph = 0, 0
    for issued in range(n_units):
        if issued >= stages:
            ok = yield from bounded_wait(cta, cta.empty[s], ph ^ 1)
            if not ok:
                break
        cta.full[s].arrive()                         # the copy lands: expect_tx completes
        s += 1
        if s == stages:
            s, ph = 0, ph ^ 1
        yield
    cta.exited.append("producer")


def mma(cta, n_units, units_per_tile, stages):
    s, fph, seg, u = 0, 0, 0, 0
    ok = True
    while u < n_units and ok:
        acc = seg & 1
        if seg >= 2:
            ok = yield from bounded_wait(cta, cta.acc_empty[acc], ((seg >> 1) & 1) ^ 1)
            if not ok:
                break
        for _ in range(min(units_per_tile, n_units - u)):
            ok = yield from bounded_wait(cta, cta.full[s], fph)
            if not ok:
                break
            cta.empty[s].arrive()                    # tcgen05.commit -> the stage is free
            s += 1
            if s == stages:
                s, fph = 0, fph ^ 1
            u += 1
            yield
        if ok:
            cta.acc_full[acc].arrive()
        seg += 1
    cta.exited.append("mma")


def epilogue(cta, n_units, units_per_tile, warp, arrives=True):
    n_seg = -(-n_units // units_per_tile)
    for seg in range(n_seg):
        acc = seg & 1
        ok = yield from bounded_wait(cta, cta.acc_full[acc], (seg >> 1) & 1)
        if not ok:
            break
        yield                                        # drain the accumulator
        if arrives:
            cta.acc_empty[acc].arrive()
    cta.exited.append(f"epilogue{warp}")


def run(n_units=23, units_per_tile=4, stages=3, silent_warp=None, max_ticks=100000):
    cta = Cta(stages)
    roles = [producer(cta, n_units, stages), mma(cta, n_units, units_per_tile, stages)]
    roles += [epilogue(cta, n_units, units_per_tile, w, arrives=(w != silent_warp)) for w in range(4)]
    live = list(roles)
    for tick in itertools.count():
        assert tick < max_ticks, "the model itself hung: a wait without a budget"
        if not live:
            break
        for r in list(live):
            try:
                next(r)
            except StopIteration:
                live.remove(r)
    cta.tmem_freed = True                            # the exit path behind __syncthreads()
    return cta, tick


def test_all_roles_finish_when_every_arrival_comes():
    cta, _ = run()
    assert cta.status == 0 and not cta.abort and cta.timeouts == 0
    assert sorted(cta.exited) == sorted(["producer", "mma"] + [f"epilogue{w}" for w in range(4)])
    assert cta.tmem_freed


def test_an_underfilled_arrival_count_expires_one_wait_and_unwinds_every_role():
    # epilogue warp 2 never releases the accumulators: acc_empty gets 3 of its 4 arrivals
    cta, ticks = run(silent_warp=2)
    assert cta.status == JK_ERR_TIMEOUT and cta.abort
    assert cta.timeouts == 1                         # one wait expired; the others saw the flag
    assert sorted(cta.exited) == sorted(["producer", "mma"] + [f"epilogue{w}" for w in range(4)])
    assert cta.tmem_freed
    assert ticks < 20 * BUDGET                       # bounded: no role outlived the budget by much


def test_the_first_error_is_kept():
    cta, _ = run(silent_warp=0)
    cta2 = Cta(2)
    cta2.status = -9                                 # an earlier bounds error
    g = bounded_wait(cta2, PhaseBarrier(1), 0)
    for _ in g:
        pass
    assert cta2.status == -9 and cta2.abort and cta.status == JK_ERR_TIMEOUT
