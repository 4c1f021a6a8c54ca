"""Deliberately naive cross-checks for the oracle (test infrastructure, tiny inputs only).

Nothing here is fast or clever: stage aggregates are built token by token, the scheduler keeps
real request objects, a real waiting list and a real free list of block ids, and selection is
all-pairs brute force.  It exists so that a slip in the oracle's aggregated formulas or in its
"the waiting queue is just an index" shortcut shows up as a disagreement.
"""
from __future__ import annotations

import math


# ---- stage aggregates, token by token (Sec. 3.2 Step 2: tasks of the prefill and decode stage) ----

def prefill_aggregates(b: int, lin: int):
    """(T, E, A, C): every prompt token is a query; each query is charged the whole prompt."""
    T = E = A = Cc = 0
    for _seq in range(b):
        E += 1
        Cc += lin                      # context the pass reads for this sequence
        for _tok in range(lin):
            T += 1
            A += lin                   # one query token x attended context
    return T, E, A, Cc


def segment_passes(sb: int, lin: int, seg: int):
    """One (T, E, A, C) per prompt segment of a sub-batch of sb requests (Sec. 3.3.2): the tokens of
    a segment attend their prompt up to the end of that segment; the last segment emits a token."""
    passes = []
    done = 0
    while done < lin:
        q = min(seg, lin - done)
        T = E = A = Cc = 0
        for _seq in range(sb):
            if done + q == lin:
                E += 1
            Cc += done + q
            for _tok in range(q):
                T += 1
                A += done + q
        passes.append((T, E, A, Cc))
        done += q
    return passes


def sub_batches(b: int, split: int):
    """Sec. 3.3.1: sub-batches of split requests, the remainder as one more."""
    out = [split] * (b // split)
    if b % split:
        out.append(b % split)
    return out


def decode_aggregates(b: int, lin: int, lout: int):
    """(T, E, A, C, R) of the whole decode stage: steps 1..Lout-1, step j attends Lin + j tokens."""
    T = E = A = Cc = R = 0
    for j in range(1, lout):
        R += 1
        for _seq in range(b):
            T += 1
            E += 1
            A += lin + j
            Cc += lin + j
    return T, E, A, Cc, R


# ---- continuous batching with explicit objects ----------------------------------------------------

class _Req:
    __slots__ = ("idx", "arrival", "lin", "lout", "gen", "cache", "blocks", "needs_prefill", "first", "finish", "todo", "seen")

    def __init__(self, idx, arrival, lin, lout):
        self.idx, self.arrival, self.lin, self.lout = idx, arrival, lin, lout
        self.gen = 0
        self.cache = 0
        self.blocks = []
        self.needs_prefill = False
        self.first = None
        self.finish = None


def trace_sim(arrival, in_len, out_len, max_batch, n_blocks, kv_block, iter_time, max_iters=10**6):
    """Prompt-priority continuous batching over paged KV with evict-youngest + recompute.

    iter_time(T, E, A, C) -> seconds of one iteration.  Returns a dict with per-request first-token
    and finish times, the makespan, decode token/time totals, iteration counts and preemptions.
    Checks as it goes that no block is owned twice and none is leaked.
    """
    reqs = [_Req(i, arrival[i], in_len[i], out_len[i]) for i in range(len(arrival))]
    waiting = list(reqs)               # FCFS: kept sorted by index
    running = []
    free = list(range(n_blocks))
    clock = 0.0
    dec_time = 0.0
    dec_tok = n_iters = n_req_iters = n_preempt = 0
    max_running = 0

    def check_blocks():
        owned = [blk for r in running for blk in r.blocks]
        assert len(owned) == len(set(owned)), "a block is owned twice"
        assert len(owned) + len(free) == n_blocks, "a block leaked"
        assert not set(owned) & set(free)
        for r in running:
            if not r.needs_prefill:
                assert len(r.blocks) == math.ceil(r.cache / kv_block)

    while True:
        # admit from the head of the queue only
        while waiting and waiting[0].arrival <= clock and len(running) < max_batch:
            r = waiting[0]
            need = math.ceil((r.lin + r.gen) / kv_block)
            if need > len(free):
                break
            r.blocks = [free.pop() for _ in range(need)]
            r.needs_prefill = True
            running.append(waiting.pop(0))
        if not running:
            if not waiting:
                break
            assert waiting[0].arrival > clock, "stuck with an empty machine"
            clock = waiting[0].arrival
            continue
        assert n_iters < max_iters
        max_running = max(max_running, len(running))
        assert [r.idx for r in running] == sorted(r.idx for r in running)
        assert all(w.idx > running[-1].idx for w in waiting)

        prompts = [r for r in running if r.needs_prefill]
        if prompts:
            T = E = A = Cc = 0
            for r in prompts:
                q = r.lin + r.gen
                E += 1
                for _ in range(q):
                    T += 1
                    A += q
                Cc += q
            dt = iter_time(T, E, A, Cc)
            after = clock + dt
            for r in prompts:
                r.cache = r.lin + r.gen
                r.gen += 1
                r.needs_prefill = False
                if r.first is None:
                    r.first = after
            part = len(prompts)
        else:
            def needers():
                return [r for r in running if r.cache % kv_block == 0]
            while len(needers()) > len(free):
                victim = max(running, key=lambda r: r.idx)
                running.remove(victim)
                free.extend(victim.blocks)
                victim.blocks = []
                victim.cache = 0
                waiting.insert(0, victim)
                assert [w.idx for w in waiting] == sorted(w.idx for w in waiting)
                n_preempt += 1
            assert running
            for r in needers():
                r.blocks.append(free.pop())
            T = E = len(running)
            A = Cc = sum(r.cache + 1 for r in running)      # cached tokens + the new one
            dt = iter_time(T, E, A, Cc)
            for r in running:
                r.cache += 1
                r.gen += 1
            dec_time = dec_time + dt
            dec_tok += len(running)
            part = len(running)
        clock = clock + dt
        n_iters += 1
        n_req_iters += part
        for r in list(running):
            if r.gen == r.lout:
                r.finish = clock
                free.extend(r.blocks)
                r.blocks = []
                running.remove(r)
        check_blocks()

    assert all(r.finish is not None and r.first is not None for r in reqs), "a request never finished"
    assert len(free) == n_blocks
    return {"first": [r.first for r in reqs], "finish": [r.finish for r in reqs], "makespan": clock,
            "dec_time": dec_time, "dec_tok": dec_tok, "n_iters": n_iters, "n_req_iters": n_req_iters,
            "n_preempt": n_preempt, "max_running": max_running}


def trace_sim_fuse(arrival, in_len, out_len, max_batch, n_blocks, kv_block, budget, iter_time, max_iters=10**6):
    """Dynamic split-and-fuse continuous batching: every iteration carries `budget` tokens, one per
    decoding request first, the rest filled with prompt tokens in arrival order (long prompts are
    spread over iterations, short ones share one).  Blocks for the whole prompt are taken at
    admission; evict-youngest + recompute as in trace_sim.  Also returns the composition of every
    iteration: (clock before, decoding request ids, [(request id, first token, q)])."""
    reqs = [_Req(i, arrival[i], in_len[i], out_len[i]) for i in range(len(arrival))]
    for r in reqs:
        r.todo = 0          # prompt tokens (and tokens to recompute) not yet processed
        r.seen = 0          # ... already processed
    waiting = list(reqs)
    running = []
    free = list(range(n_blocks))
    clock = 0.0
    dec_time = 0.0
    dec_tok = n_iters = n_req_iters = n_preempt = 0
    log = []
    while True:
        while waiting and waiting[0].arrival <= clock and len(running) < max_batch:
            r = waiting[0]
            need = math.ceil((r.lin + r.gen) / kv_block)
            if need > len(free):
                break
            r.blocks = [free.pop() for _ in range(need)]
            r.todo, r.seen = r.lin + r.gen, 0
            running.append(waiting.pop(0))
        if not running:
            if not waiting:
                break
            assert waiting[0].arrival > clock, "stuck with an empty machine"
            clock = waiting[0].arrival
            continue
        assert n_iters < max_iters
        assert [r.idx for r in running] == sorted(r.idx for r in running)

        def needers():
            return [r for r in running if r.todo == 0 and r.cache % kv_block == 0]
        while len(needers()) > len(free):
            victim = max(running, key=lambda r: r.idx)
            running.remove(victim)
            free.extend(victim.blocks)
            victim.blocks, victim.cache, victim.todo, victim.seen = [], 0, 0, 0
            waiting.insert(0, victim)
            n_preempt += 1
        assert running
        for r in needers():
            r.blocks.append(free.pop())
        decoders = [r for r in running if r.todo == 0]
        # decoders come before requests still in their prompt (arrival order, oldest served first)
        assert [r.idx for r in running] == [r.idx for r in decoders] + [r.idx for r in running if r.todo > 0]
        T = E = A = Cc = 0
        for r in decoders:
            T += 1
            E += 1
            A += r.cache + 1
            Cc += r.cache + 1
        left = max(0, budget - len(decoders))
        chunks = []
        for r in running:
            if r.todo == 0 or left == 0:
                continue
            q = min(r.todo, left)
            for _ in range(q):
                T += 1
                A += r.seen + q             # every token of the chunk attends the prompt up to the chunk's end
            Cc += r.seen + q
            if q == r.todo:
                E += 1
            chunks.append((r, q))
            left -= q
        assert T > 0 and T <= max(budget, len(decoders))
        dt = iter_time(T, E, A, Cc)
        log.append((clock, [r.idx for r in decoders], [(r.idx, r.seen, q) for r, q in chunks]))
        after = clock + dt
        for r in decoders:
            r.cache += 1
            r.gen += 1
        for r, q in chunks:
            r.seen += q
            r.todo -= q
            if r.todo == 0:
                r.cache = r.lin + r.gen
                r.gen += 1
                if r.first is None:
                    r.first = after
        if decoders:
            dec_time = dec_time + dt
            dec_tok += len(decoders)
        clock = after
        n_iters += 1
        n_req_iters += len(decoders) + len(chunks)
        for r in list(running):
            if r.todo == 0 and r.gen == r.lout:
                r.finish = clock
                free.extend(r.blocks)
                r.blocks = []
                running.remove(r)
        owned = [blk for r in running for blk in r.blocks]
        assert len(owned) == len(set(owned)) and len(owned) + len(free) == n_blocks
        for r in running:
            if r.todo == 0:
                assert len(r.blocks) == math.ceil(r.cache / kv_block)
    assert all(r.finish is not None and r.first is not None for r in reqs), "a request never finished"
    assert len(free) == n_blocks
    return {"first": [r.first for r in reqs], "finish": [r.finish for r in reqs], "makespan": clock,
            "dec_time": dec_time, "dec_tok": dec_tok, "n_iters": n_iters, "n_req_iters": n_req_iters,
            "n_preempt": n_preempt, "log": log}


# ---- selection by brute force ----------------------------------------------------------------------

def topk_bruteforce(keys, passing, k):
    """k times: scan for the smallest (key, index) not yet taken."""
    taken = []
    for _ in range(k):
        best = None
        for i, (v, ok) in enumerate(zip(keys, passing)):
            if not ok or i in taken:
                continue
            if best is None or v < keys[best] or (v == keys[best] and i < best):
                best = i
        if best is None:
            break
        taken.append(best)
    return taken


def pareto_bruteforce(xs, ys, passing):
    """All-pairs dominance; equal points keep the lowest index; ascending x."""
    front = []
    n = len(xs)
    for i in range(n):
        if not passing[i]:
            continue
        beaten = False
        for j in range(n):
            if j == i or not passing[j]:
                continue
            if xs[j] <= xs[i] and ys[j] <= ys[i] and (xs[j] < xs[i] or ys[j] < ys[i]):
                beaten = True
                break
            if xs[j] == xs[i] and ys[j] == ys[i] and j < i:
                beaten = True
                break
        if not beaten:
            front.append(i)
    front.sort(key=lambda i: (xs[i], ys[i], i))
    return front
