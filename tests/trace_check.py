"""Replay checker for one client's iteration trace (pure Python, small cases).

Walks a trace record by record, keeping the state the paper's rules talk about
(which requests are running, their KV lengths, the decode time waited since
the last prefill) and asserts that every record is what the rules force:

* stages are exclusive: a record is either a prefill of a queue prefix or one
  decode token for every running request (PD competition);
* every request is prefilled exactly once, before its first decode token, and
  decodes exactly o_i tokens on the client that prefilled it;
* the batch cap and the KV budget (p+o, or a fixed amount per request when the
  output length is not known at admission, reserved from admission to
  retirement) are never exceeded; admission takes the longest admissible queue prefix;
* each decision follows "prefill iff lambda * C_d > C_p" unless forced
  (nothing admissible -> decode, nothing running -> prefill);
* every duration is recomputable from its own record.

It shares no code with the oracle or the CUDA library.
"""
from __future__ import annotations

PREFILL_FLAG = 1 << 31


def replay(queue, p, o, cm, cap, kv_budget, lambda_q16, trace, kv_reserve=0):
    ap, bp, ad, bd, q = (int(x) for x in cm[:5])
    levels = [(int(a), int(b)) for a, b in cm[7]] if len(cm) > 7 else []

    def prefill_cost(tokens):              # Eq. 5-7: smallest level that holds the tokens
        if not levels:
            return ap + bp * tokens
        return next(t for c_, t in levels if tokens <= c_)
    queue = [int(i) for i in queue]
    holds = (lambda i: kv_reserve) if kv_reserve else (lambda i: int(p[i]) + int(o[i]))
    running = {}                      # request -> [kv, remaining]
    head = 0
    waited = 0                        # C_d
    clock = busy = n_pre = n_dec = 0
    sum_prefill_tokens = sum_decode_active = sum_decode_kv = 0
    decoded = {i: 0 for i in queue}
    for k, rec in enumerate(trace):
        dur, kind_n, tokens, aux = (int(x) for x in rec)
        reserved = sum(holds(i) for i in running)
        assert len(running) <= cap and reserved <= kv_budget
        # admissible prefix of the queue
        cand, extra = [], 0
        while head + len(cand) < len(queue) and len(running) + len(cand) < cap:
            i = queue[head + len(cand)]
            need = holds(i)
            if reserved + extra + need > kv_budget:
                break
            if levels and sum(int(p[x]) for x in cand) + int(p[i]) > levels[-1][0]:
                break
            cand.append(i)
            extra += need
        cp = prefill_cost(sum(int(p[i]) for i in cand))
        wants_prefill = lambda_q16 * waited > (cp << 16)
        if kind_n & PREFILL_FLAG:
            assert cand, f"record {k}: prefill with nothing admissible"
            assert not running or wants_prefill, f"record {k}: prefill against the rule"
            assert kind_n == (PREFILL_FLAG | len(cand)) and tokens == sum(int(p[i]) for i in cand)
            assert aux == head and dur == cp
            for i in cand:
                assert i not in running and decoded[i] == 0
                running[i] = [int(p[i]), int(o[i])]
            head += len(cand)
            busy += dur * len(cand)
            waited = 0
            n_pre += 1
            sum_prefill_tokens += tokens
        else:
            assert running, f"record {k}: decode with an empty batch"
            assert not cand or not wants_prefill, f"record {k}: decode against the rule"
            B, S = len(running), sum(v[0] for v in running.values())
            assert kind_n == B and tokens == S and dur == ad + bd * B + S // q
            gone = []
            for i, v in running.items():
                v[0] += 1
                v[1] -= 1
                decoded[i] += 1
                if v[1] == 0:
                    gone.append(i)
            for i in gone:
                del running[i]
            assert aux == len(gone)
            busy += dur * B
            waited = min(waited + dur, 2 ** 31 - 1)
            n_dec += 1
            sum_decode_active += B
            sum_decode_kv += S
        clock += dur
    assert head == len(queue) and not running, "trace ends before the work does"
    assert all(decoded[i] == int(o[i]) for i in queue)
    # conservation laws
    assert sum_prefill_tokens == sum(int(p[i]) for i in queue)
    assert sum_decode_active == sum(int(o[i]) for i in queue)
    assert sum_decode_kv == sum(int(o[i]) * int(p[i]) + int(o[i]) * (int(o[i]) - 1) // 2 for i in queue)
    return dict(makespan_us=clock, busy_slot_us=busy, n_prefill_iters=n_pre, n_decode_iters=n_dec)


HASH_INIT = 0xCBF29CE484222325
HASH_C = (1, 0x9E3779B1, 0x85EBCA77, 0xC2B2AE3D)
HASH_M = 0x27D4EB2F


def trace_hash(trace):
    """h <- (h + dur + C1*kind_n + C2*tokens + C3*aux) * M  (mod 2^64) per record, from h = INIT."""
    mask = (1 << 64) - 1
    h = HASH_INIT
    for rec in trace:
        h = ((h + sum(c * int(x) for c, x in zip(HASH_C, rec))) * HASH_M) & mask
    return h
