"""A host-side model of the chunk-scan kernel's mbarrier protocol (no GPU).

The kernel's roles (three TMA producers, the MMA issuer, two mask groups, two epilogue groups) talk
through phase barriers that are polled by parity.  A parity poll is only sound while the barrier is
at most one phase ahead of the waiter: two phases ahead it blocks for good, three ahead it passes
on stale data.  This model re-states the protocol (ring indices, parities, arrival counts) as the
kernel header describes it, runs it as a discrete-event simulation under many random and extreme
role speeds, decides every wait by the parity rule alone, and checks against the true phase counts
that no wait is ever lapped, that none passes early, and that every role finishes.  It also shows
that the tempting variant in which the epilogue takes the row scalars through the CBq buffer's mask
barrier does get lapped when the mask is fast.
The FP16-operand kernel's protocol (build_f16) is modelled the same way, with the variant that gave
its two MMA issuers a single barrier pair on the Cq/hq buffer as the counter-example.
"""
import heapq
import random

import pytest


class Bar:
    def __init__(self, name, count):
        self.name, self.count, self.pending, self.completed = name, count, count, 0

    def arrive(self, k=1):
        for _ in range(k):
            self.pending -= 1
            assert self.pending >= 0, f"{self.name}: more arrivals than the count of a phase"
            if self.pending == 0:
                self.completed += 1
                self.pending = self.count

    def poll(self, parity, want):
        """Hardware rule: true iff the phase of that parity has completed.  `want` is the number of
        completed phases the waiter really needs (model-side truth, for the checks only)."""
        assert self.completed <= want, f"{self.name}: lapped (completed {self.completed}, waiter needs {want})"
        ok = (self.completed & 1) != parity
        assert ok == (self.completed >= want), f"{self.name}: parity rule and phase count disagree"
        return ok


class Sim:
    """Roles are generators yielding ('wait', bar, parity, want) | ('work', t) | ('arrive', bar, k)
    | ('async', t, [(bar, k), ...]) (arrivals that happen t later: a TMA load landing, an MMA commit)."""

    def __init__(self, seed):
        self.rng = random.Random(seed)
        self.now = 0.0
        self.events = []   # (time, seq, kind, payload)
        self.seq = 0
        self.blocked = {}  # role name -> (gen, wait tuple)
        self.live = 0

    def push(self, t, kind, payload):
        self.seq += 1
        heapq.heappush(self.events, (t, self.seq, kind, payload))

    def spawn(self, name, gen):
        self.live += 1
        self.push(0.0, "run", (name, gen))

    def step_role(self, name, gen):
        while True:
            try:
                op = next(gen)
            except StopIteration:
                self.live -= 1
                return
            if op[0] == "work":
                self.push(self.now + op[1], "run", (name, gen))
                return
            if op[0] == "arrive":
                op[1].arrive(op[2])
                self.wake()
            elif op[0] == "async":
                self.push(self.now + op[1], "arrivals", op[2])
            elif op[0] == "wait":
                if not op[1].poll(op[2], op[3]):
                    self.blocked[name] = (gen, op)
                    return

    def wake(self):
        for name in list(self.blocked):
            gen, op = self.blocked[name]
            if op[1].poll(op[2], op[3]):
                del self.blocked[name]
                self.push(self.now, "run", (name, gen))

    def run(self):
        while self.events:
            self.now, _, kind, payload = heapq.heappop(self.events)
            if kind == "run":
                self.step_role(*payload)
            else:
                for bar, k in payload:
                    bar.arrive(k)
                self.wake()
        assert self.live == 0 and not self.blocked, f"deadlock: blocked {sorted(self.blocked)}"


def build(sim, ntiles, ntpu, speed, epilogue_waits_on_mq=False):
    rng = sim.rng
    B = lambda name, count, n: [Bar(f"{name}{i}", count) for i in range(n)]
    cb_full, cb_free, mq = B("CB_FULL", 1, 4), B("CB_FREE", 1, 4), B("MQ", 8, 4)
    tok_full, tok_free = B("TOK_FULL", 1, 4), B("TOK_FREE", 8, 4)
    acc, acc_free = B("ACC", 1, 4), B("ACC_FREE", 4, 4)
    row_full, row_free = B("ROW_FULL", 9, 8), B("ROW_FREE", 4, 8)
    ch_full, ch_free = Bar("CH_FULL", 1), Bar("CH_FREE", 1)
    x_full, x_free = B("X_FULL", 1, 2), B("X_FREE", 4 if ntpu == 1 else 8, 2)

    it_of = lambda n: n % ntpu
    cb_index = lambda n: (n & 3) if ntpu == 1 else ((0 if it_of(n) else 2) + ((n >> 1) & 1))
    cb_use = lambda n: (n >> 2)                       # how often tile n's CBq buffer was used before
    x_index = lambda n: (n & 1) if ntpu == 1 else ((n >> 1) & 1)
    x_use = lambda n: (n >> 1) if ntpu == 1 else (n >> 2)
    x_phase = lambda n: x_use(n) & 1
    t = lambda role: rng.expovariate(1.0) * speed[role]
    full = lambda bar, use: ("wait", bar, use & 1, use + 1)          # phase `use` of the barrier has completed
    free = lambda bar, use: ("wait", bar, (use & 1) ^ 1, use)        # its phase use - 1 has (none for use = 0)

    def prod_cb():
        for n in range(ntiles):
            ci, t3, r8 = cb_index(n), n & 3, n & 7
            yield free(cb_free[ci], cb_use(n))
            yield ("async", t("load"), [(cb_full[ci], 1)])
            yield free(tok_free[t3], n >> 2)
            yield ("async", t("load"), [(tok_full[t3], 1)])
            yield free(row_free[r8], n >> 3)
            yield ("async", t("load"), [(row_full[r8], 1)])
            yield ("work", t("producer"))

    def prod_ch():
        for n in range(ntiles):
            yield free(ch_free, n)
            yield ("async", t("load"), [(ch_full, 1)])
            yield ("work", t("producer"))

    def prod_x():
        for n in range(ntiles):
            if it_of(n) == 0:
                yield free(x_free[x_index(n)], x_use(n))
                yield ("async", t("load"), [(x_full[x_index(n)], 1)])
            yield ("work", t("producer"))

    def mma():
        for n in range(ntiles):
            ci, a4, xs = cb_index(n), n & 3, x_index(n)
            yield free(acc_free[a4], n >> 2)
            yield full(ch_full, n)
            yield ("work", t("mma"))
            yield ("async", t("mma"), [(ch_free, 1)])
            yield full(mq[ci], cb_use(n))
            yield full(x_full[xs], x_use(n))
            yield ("work", t("mma"))
            yield ("async", t("mma"), [(cb_free[ci], 1), (acc[a4], 1)])

    def mask(g):
        for n in range(ntiles):
            if (((n if ntpu == 1 else n >> 1)) & 1) != g:
                continue
            ci, t3, r8 = cb_index(n), n & 3, n & 7
            yield full(tok_full[t3], n >> 2)
            yield full(cb_full[ci], cb_use(n))
            yield free(row_free[r8], n >> 3)
            yield ("work", t("mask") * (1 + 2 * it_of(n)))
            yield ("arrive", mq[ci], 8)
            yield ("arrive", tok_free[t3], 8)
            yield ("arrive", row_full[r8], 8)

    def epilogue(eg):
        for n in range(eg, ntiles, 2):
            a4, xs, r8 = n & 3, x_index(n), n & 7
            yield full(acc[a4], n >> 2)
            if epilogue_waits_on_mq:
                yield full(mq[cb_index(n)], cb_use(n))
            yield full(x_full[xs], x_use(n))
            yield full(row_full[r8], n >> 3)
            yield ("work", t("epilogue"))
            yield ("arrive", acc_free[a4], 4)
            yield ("arrive", x_free[xs], 4)
            yield ("arrive", row_free[r8], 4)

    for name, gen in [("prod_cb", prod_cb()), ("prod_ch", prod_ch()), ("prod_x", prod_x()), ("mma", mma()),
                      ("mask0", mask(0)), ("mask1", mask(1)), ("epi0", epilogue(0)), ("epi1", epilogue(1))]:
        sim.spawn(name, gen)


def build_f16(sim, ntiles, ntpu, speed, one_ch_barrier=False):
    """The FP16-operand kernel: one epilogue group of eight warps that also hands back the scalar pack,
    two MMA issuers on alternate tiles with a barrier pair each on the single Cq/hq buffer, operand buffers
    in tensor memory released by the MMA, and xq codes requested by the epilogue when it frees a buffer
    and expanded to FP16 by the mask group that takes the chunk."""
    rng = sim.rng
    B = lambda name, count, n: [Bar(f"{name}{i}", count) for i in range(n)]
    cb_full, cb_free, mq = B("CB_FULL", 1, 4), B("CB_FREE", 8, 4), B("MQ", 8, 4)
    tok_full, tok_free = B("TOK_FULL", 1, 4), B("TOK_FREE", 8, 4)
    acc, acc_free, afree = B("ACC", 1, 2), B("ACC_FREE", 8, 2), B("AFREE", 1, 2)
    ch_full, ch_free = B("CH_FULL", 1, 2), B("CH_FREE", 1, 2)
    x_raw, x_full, x_free = B("X_RAW", 1, 2), B("X_FULL", 8, 2), B("X_FREE", 8 * ntpu, 2)

    it_of = lambda n: n % ntpu
    cb_index = lambda n: (n & 3) if ntpu == 1 else ((0 if it_of(n) else 2) + ((n >> 1) & 1))
    cb_use = lambda n: (n >> 2)
    x_index = lambda n: (n & 1) if ntpu == 1 else ((n >> 1) & 1)
    x_use = lambda n: (n >> 1) if ntpu == 1 else (n >> 2)
    t = lambda role: rng.expovariate(1.0) * speed[role]
    full = lambda bar, use: ("wait", bar, use & 1, use + 1)
    free = lambda bar, use: ("wait", bar, (use & 1) ^ 1, use)

    def prod_cb():
        for kc in range(2):                                   # the codes of the first two chunks
            if kc * ntpu < ntiles:
                yield ("async", t("load"), [(x_raw[kc], 1)])
        for n in range(ntiles):
            ci, t3 = cb_index(n), n & 3
            yield free(cb_free[ci], cb_use(n))
            yield ("async", t("load"), [(cb_full[ci], 1)])
            yield free(tok_free[t3], n >> 2)
            yield ("async", t("load"), [(tok_full[t3], 1)])
            yield ("work", t("producer"))

    def prod_ch():
        for n in range(ntiles):
            if one_ch_barrier:
                yield free(ch_free[0], n)
                yield ("async", t("load"), [(ch_full[0], 1)])
            else:
                if n > 0:
                    yield full(ch_free[(n - 1) & 1], (n - 1) >> 1)   # the other issuer's MMAs have read the buffer
                yield ("async", t("load"), [(ch_full[n & 1], 1)])
            yield ("work", t("producer"))

    def issuer(par):
        for n in range(par, ntiles, 2):
            ci, s2, xs = cb_index(n), n & 1, x_index(n)
            yield free(acc_free[s2], n >> 1)
            yield full(ch_full[0], n) if one_ch_barrier else full(ch_full[par], n >> 1)
            yield ("work", t("mma"))
            yield ("async", t("mma"), [(ch_free[0 if one_ch_barrier else par], 1)])
            yield full(mq[ci], cb_use(n))
            yield full(x_full[xs], x_use(n))
            yield ("work", t("mma"))
            yield ("async", t("mma"), [(afree[s2], 1), (acc[s2], 1)])

    def mask(g):
        for n in range(ntiles):
            if (((n if ntpu == 1 else n >> 1)) & 1) != g:
                continue
            ci, t3, ob, xs = cb_index(n), n & 3, n & 1, x_index(n)
            yield full(tok_full[t3], n >> 2)
            yield full(cb_full[ci], cb_use(n))
            yield free(afree[ob], n >> 1)
            if it_of(n) == 0:
                yield full(x_raw[xs], x_use(n))
                yield ("work", t("mask") * 0.2)
                yield ("arrive", x_full[xs], 8)
            yield ("work", t("mask") * (1 + 2 * it_of(n)))
            yield ("arrive", mq[ci], 8)
            yield ("arrive", cb_free[ci], 8)

    def epilogue():
        for n in range(ntiles):
            s2, xs, t3 = n & 1, x_index(n), n & 3
            yield full(acc[s2], n >> 1)
            yield full(x_full[xs], x_use(n))
            yield full(tok_full[t3], n >> 2)
            yield ("work", t("epilogue"))
            yield ("arrive", acc_free[s2], 8)
            yield ("arrive", x_free[xs], 8)
            yield ("arrive", tok_free[t3], 8)
            if it_of(n) == ntpu - 1 and n - (ntpu - 1) + 2 * ntpu < ntiles:
                yield full(x_free[xs], x_use(n))               # every warp is through with the chunk
                yield ("async", t("load"), [(x_raw[xs], 1)])   # the codes of the chunk after next

    for name, gen in [("prod_cb", prod_cb()), ("prod_ch", prod_ch()), ("mma0", issuer(0)), ("mma1", issuer(1)),
                      ("mask0", mask(0)), ("mask1", mask(1)), ("epi", epilogue())]:
        sim.spawn(name, gen)


SPEEDS = [
    dict(load=1.0, producer=0.1, mma=0.3, mask=2.0, epilogue=2.0),     # roughly the measured ratios
    dict(load=1.0, producer=0.1, mma=0.3, mask=0.01, epilogue=5.0),    # instant mask, slow epilogue
    dict(load=1.0, producer=0.1, mma=0.3, mask=5.0, epilogue=0.01),    # slow mask, instant epilogue
    dict(load=10.0, producer=0.01, mma=0.01, mask=0.1, epilogue=0.1),  # slow memory
    dict(load=0.01, producer=0.01, mma=5.0, mask=0.1, epilogue=0.1),   # slow MMA issue
    dict(load=0.01, producer=5.0, mma=0.01, mask=0.01, epilogue=0.01), # slow producers
]


@pytest.mark.parametrize("ntpu", [1, 2])
@pytest.mark.parametrize("speed", range(len(SPEEDS)))
def test_no_wait_is_lapped_and_every_role_finishes(ntpu, speed):
    for seed in range(20):
        sim = Sim(1000 * speed + seed)
        build(sim, ntiles=36, ntpu=ntpu, speed=SPEEDS[speed])
        sim.run()


def test_a_mask_barrier_wait_in_the_epilogue_would_be_lapped():
    """The CBq buffer's mask barrier may complete for tile n + 4 while the epilogue group that owns tile
    n is still busy with tile n - 2: nothing the epilogue releases stands between the two."""
    hit = 0
    for seed in range(20):
        sim = Sim(seed)
        build(sim, ntiles=36, ntpu=2, speed=SPEEDS[1], epilogue_waits_on_mq=True)
        try:
            sim.run()
        except AssertionError as e:
            assert "MQ" in str(e) or "deadlock" in str(e)
            hit += 1
    assert hit > 0


@pytest.mark.parametrize("ntpu", [1, 2])
@pytest.mark.parametrize("speed", range(len(SPEEDS)))
def test_fp16_operand_kernel_protocol(ntpu, speed):
    for seed in range(20):
        sim = Sim(5000 + 1000 * speed + seed)
        build_f16(sim, ntiles=36, ntpu=ntpu, speed=SPEEDS[speed])
        sim.run()


def test_two_issuers_on_one_barrier_pair_would_pass_a_wait_early():
    """With a single barrier pair on the Cq/hq buffer, the issuer of the odd tiles polls the parity of
    phase 1 before phase 0 has completed, which a fresh barrier answers with yes."""
    with pytest.raises(AssertionError, match="CH_FULL"):
        sim = Sim(1)
        build_f16(sim, ntiles=36, ntpu=2, speed=SPEEDS[0], one_ch_barrier=True)
        sim.run()

