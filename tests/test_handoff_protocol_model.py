"""Host-side model of the barrier protocol of the spare-buffer fused kernel (fused4s_kernel.cuh).

The kernel hands score buffers round between T query tiles through mbarriers whose waits are PARITY waits:
`wait(parity)` returns as soon as the barrier's current phase has the other parity, so it is only sound for a
waiter exactly one phase behind.  This model runs the same roles (TMA producer, one MMA issuer per tile, the
softmax warps, an in-order tensor pipe) as coroutines under a random scheduler, with barriers that have exactly
that semantics, and checks that nothing deadlocks and that every read sees the contents it expects (the right
score tile, the right weights, the right K/V stage).  A per-buffer barrier (instead of one per tile and buffer)
fails here within a few schedules -- on the GPU it showed as expired waits.
"""
import random

import pytest


class Bar:
    def __init__(self, count):
        self.count, self.pending, self.phase = count, count, 0

    def arrive(self):
        self.pending -= 1
        assert self.pending >= 0
        if self.pending == 0:
            self.phase += 1
            self.pending = self.count

    def done(self, parity):   # mbarrier.try_wait.parity
        return (self.phase & 1) != parity


def simulate(T, n_kv, stages, seed, warps=4, per_tile_barriers=True, limit=400000):
    rnd = random.Random(seed)
    NB = T + 1
    nt = 4 if per_tile_barriers else 1
    s_full = [[Bar(1) for _ in range(5)] for _ in range(nt)]
    p_full = [[Bar(warps) for _ in range(5)] for _ in range(nt)]
    sel = (lambda t: t) if per_tile_barriers else (lambda t: 0)
    q_full = [Bar(1) for _ in range(4)]
    pv_done = [Bar(1) for _ in range(4)]
    o_final = [Bar(1) for _ in range(4)]
    kv_full = [Bar(1) for _ in range(stages)]
    kv_empty = [Bar(T) for _ in range(stages)]
    pipe, buf, stage, errors = [], {}, {}, []

    def check(cond, what):
        if not cond:
            errors.append(what)

    def producer():
        for t in range(T):
            q_full[t].arrive()
        yield
        for j in range(n_kv):
            s = j % stages
            if j >= stages:
                while not kv_empty[s].done(((j // stages) - 1) & 1):
                    yield
            stage[s] = j
            kv_full[s].arrive()
            yield

    def issuer(t):
        tn = 0 if t + 1 == T else t + 1
        while not (kv_full[0].done(0) and q_full[t].done(0) and q_full[tn].done(0)):
            yield

        def issue_s(tile, j, b):
            check(stage.get(j % stages) == j, ("S reads a stale stage", tile, j))
            pipe.append(("S", tile, j, b, [s_full[sel(tile)][b]]))
        issue_s(t, 0, t)
        if t == T - 1 and n_kv > 1:
            while not kv_full[1 % stages].done((1 // stages) & 1):
                yield
            issue_s(tn, 1, T)
        b, ph, jm = t, 0, 0
        for j in range(n_kv):
            jn = j + (2 if t + 1 == T else 1)
            more = jn < n_kv
            if more:
                while not kv_full[jn % stages].done((jn // stages) & 1):
                    yield
            while not p_full[sel(t)][b].done(ph):
                yield
            check(stage.get(j % stages) == j, ("P V reads a stale stage", t, j))
            check(buf.get(b) == ("P", t, j), ("P V reads the wrong weights", t, j, b, buf.get(b)))
            pipe.append(("PV", t, j, b, []))
            if more:
                issue_s(tn, jn, b)
            pipe.append(("C", t, j, b, [pv_done[t], kv_empty[j % stages]] + ([o_final[t]] if j == n_kv - 1 else [])))
            b = NB - 1 if b == 0 else b - 1
            jm += 1
            if jm == NB:
                jm, ph = 0, ph ^ 1
            yield

    def softmax(t):
        b, ph, jm = t % NB, 0, 0
        for j in range(n_kv):
            while not s_full[sel(t)][b].done(ph):
                yield
            check(buf.get(b) in (("S", t, j), ("P", t, j)), ("softmax reads the wrong scores", t, j, b, buf.get(b)))
            yield
            buf[b] = ("P", t, j)
            if j > 0:
                while not pv_done[t].done((j - 1) & 1):
                    yield
            p_full[sel(t)][b].arrive()
            b = NB - 1 if b == 0 else b - 1
            jm += 1
            if jm == NB:
                jm, ph = 0, ph ^ 1
            yield
        while not o_final[t].done(0):
            yield

    procs = [producer()] + [issuer(t) for t in range(T)] + [softmax(t) for t in range(T) for _ in range(warps)]
    steps = 0
    while procs and not errors:
        steps += 1
        if steps > limit:
            return "deadlock"
        if pipe and rnd.random() < 0.5:      # the tensor pipe retires its queue in order
            kind, tile, j, b, bars = pipe.pop(0)
            if kind == "S":
                buf[b] = ("S", tile, j)
            for x in bars:
                x.arrive()
        i = rnd.randrange(len(procs))
        try:
            next(procs[i])
        except StopIteration:
            procs.pop(i)
    return errors[0] if errors else "ok"


@pytest.mark.parametrize("T", [1, 2, 3, 4])
@pytest.mark.parametrize("n_kv", [1, 2, 3, 8, 9, 17])
def test_rotation_protocol_completes_with_the_right_contents(T, n_kv):
    for seed in range(3):
        assert simulate(T, n_kv, 8, seed) == "ok"


def test_one_barrier_per_buffer_is_not_enough():
    """Different tiles consuming successive phases of ONE barrier per buffer can start waiting a phase early."""
    outcomes = {simulate(4, 17, 8, seed, per_tile_barriers=False) for seed in range(12)}
    assert outcomes != {"ok"}


# ---------------------------------------------------------------------------------------------------------------
# The variant for ONE query tile per CTA: the key tiles are dealt out among SPLIT warpgroups ("parts": part g takes
# key tiles g, g + SPLIT, ...), NB score buffers run ahead of the products, and the MMAs come from TWO threads -- the
# products O_g (+)= P(j) V(j) from one, the scores of key tile j + NB from the other -- whose instructions the tensor
# pipe does not order against each other.

def simulate_parts(SPLIT, NB, n_kv, stages, seed, warps=4, wait_buf_free=True, limit=400000):
    rnd = random.Random(seed)
    s_full = [Bar(1) for _ in range(NB)]
    p_full = [Bar(warps) for _ in range(NB)]
    buf_free = [Bar(1) for _ in range(NB)]
    pv_done = [Bar(1) for _ in range(SPLIT)]
    o_final = Bar(1)
    q_full = Bar(1)
    kv_full = [Bar(1) for _ in range(stages)]
    kv_empty = [Bar(1) for _ in range(stages)]
    pipe_a, pipe_b = [], []                      # per issuing thread, each retired in order
    buf = {b: {} for b in range(NB)}             # per buffer and warp: what it holds
    stage, errors = {}, []

    def check(cond, what):
        if not cond:
            errors.append(what)

    def producer():
        q_full.arrive()
        yield
        for j in range(n_kv):
            s = j % stages
            if j >= stages:
                while not kv_empty[s].done(((j // stages) - 1) & 1):
                    yield
            stage[s] = j
            kv_full[s].arrive()
            yield

    def score_thread():
        while not q_full.done(0):
            yield
        for jn in range(n_kv):
            b = jn % NB
            while not kv_full[jn % stages].done((jn // stages) & 1):
                yield
            if jn >= NB and wait_buf_free:
                while not buf_free[b].done(((jn // NB) - 1) & 1):
                    yield
            check(stage.get(jn % stages) == jn, ("S reads a stale stage", jn))
            pipe_b.append(("S", jn, b, [s_full[b]]))
            yield

    def product_thread():
        for j in range(n_kv):
            b = j % NB
            while not p_full[b].done((j // NB) & 1):
                yield
            check(stage.get(j % stages) == j, ("P V reads a stale stage", j))
            pipe_a.append(("PV", j, b, [pv_done[j % SPLIT], buf_free[b], kv_empty[j % stages]] +
                           ([o_final] if j == n_kv - 1 else [])))
            yield

    def part_warp(g, w):
        for i, j in enumerate(range(g, n_kv, SPLIT)):
            b = j % NB
            while not s_full[b].done((j // NB) & 1):
                yield
            check(buf[b].get(w) == ("S", j), ("a part reads the wrong scores", g, w, j, b, buf[b].get(w)))
            yield
            buf[b][w] = ("P", j)
            if i > 0:          # the product of the part's previous key tile
                while not pv_done[g].done((i - 1) & 1):
                    yield
            p_full[b].arrive()
            yield
        while not o_final.done(0):
            yield

    procs = [producer(), score_thread(), product_thread()] + [part_warp(g, w) for g in range(SPLIT) for w in range(warps)]
    steps = 0
    while procs and not errors:
        steps += 1
        if steps > limit:
            return "deadlock"
        for pipe in (pipe_a, pipe_b):        # two in-order queues, retired independently of one another
            if pipe and rnd.random() < 0.4:
                kind, j, b, bars = pipe.pop(0)
                if kind == "S":
                    for w in range(warps):
                        buf[b][w] = ("S", j)
                else:
                    check(all(buf[b].get(w) == ("P", j) for w in range(warps)), ("P V reads the wrong weights", j, b))
                for x in bars:
                    x.arrive()
        i = rnd.randrange(len(procs))
        try:
            next(procs[i])
        except StopIteration:
            procs.pop(i)
    return errors[0] if errors else "ok"


@pytest.mark.parametrize("SPLIT,NB", [(2, 2), (2, 4), (4, 4)])
@pytest.mark.parametrize("n_kv", [1, 2, 3, 4, 5, 8, 16, 17])
def test_lone_tile_in_parts_protocol(SPLIT, NB, n_kv):
    for seed in range(4):
        assert simulate_parts(SPLIT, NB, n_kv, 8, seed) == "ok"
        assert simulate_parts(SPLIT, NB, n_kv, NB + 1, seed) == "ok"


def test_scores_must_wait_for_the_completion_of_the_products_they_overwrite():
    """Without the per-buffer completion barrier the second thread's scores can land on weights not yet read."""
    outcomes = {simulate_parts(2, 4, 17, 8, seed, wait_buf_free=False) for seed in range(12)}
    assert outcomes != {"ok"}
