"""Timeline of the three attention routes of Section 3.3 under a synthetic input arrival process.

The paper's latency tables (Section 4.1, "Metric"; Appendix F) let the input arrive at a fixed speaking rate
(150 words per minute) and compare three routes:

* batch       : one cache; reasoning starts when the whole input has arrived and has been prefilled;
* interleaved : one cache; input units and reasoning units alternate, so the next input unit cannot be
                encoded while the model reasons about the current one;
* streaming   : two caches; prefill of unit u + 1 runs beside the reasoning about unit u (Algorithm 1).

This module holds no attention arithmetic and launches nothing: it is a discrete-event calculation on
per-call durations that the caller measured (or assumes), and it reports the paper's quantities -- input tokens
consumed before the first reasoning token, time of the first reasoning token, delay between the end of the
input and the end of the reasoning.
"""
from __future__ import annotations

from dataclasses import dataclass

WORDS_PER_MINUTE = 150.0       # the paper's speaking rate
TOKENS_PER_WORD = 1.3          # assumption of this build: sub-word tokens per word


@dataclass
class RouteTimeline:
    route: str
    ttft_tokens: int           # input tokens that had to arrive before the first reasoning token
    first_token_s: float       # time of the first reasoning token, from the start of the input
    input_end_s: float         # arrival time of the last input token
    done_s: float              # time of the last reasoning token
    delay_s: float             # done_s - input_end_s: what the user waits after having finished speaking


def arrival_times(src_unit_len, tokens_per_second):
    """Arrival time of the last token of every input unit."""
    t, out = 0.0, []
    for n in src_unit_len:
        t += n / tokens_per_second
        out.append(t)
    return out


def simulate(route, src_unit_len, rsn_unit_len, final_len, prefill_s, decode_step_s, tokens_per_second=None):
    """prefill_s(u, n_units_at_once) -> seconds of one prefill call that encodes input units u .. u+n-1;
    decode_step_s(r) -> seconds of the decode step that produces reasoning token r (0-based)."""
    rate = tokens_per_second or WORDS_PER_MINUTE / 60.0 * TOKENS_PER_WORD
    U = len(src_unit_len)
    arrive = arrival_times(src_unit_len, rate)
    input_end = arrive[-1] if U else 0.0
    r = 0                     # reasoning tokens produced
    first = None
    ttft = 0

    def decode(t, count):
        nonlocal r, first
        for _ in range(count):
            t += decode_step_s(r)
            if first is None:
                first = t
            r += 1
        return t

    if route == "batch":
        t = input_end + (prefill_s(0, U) if U else 0.0)
        ttft = sum(src_unit_len)
        for u in range(U):
            t = decode(t, rsn_unit_len[u])
        t = decode(t, final_len)
    elif route == "interleaved":
        t = 0.0
        for u in range(U):
            t = max(t, arrive[u]) + prefill_s(u, 1)     # the one cache is busy while the model reasons
            if first is None and (rsn_unit_len[u] > 0):
                ttft = sum(src_unit_len[: u + 1])
            t = decode(t, rsn_unit_len[u])
        if first is None:
            ttft = sum(src_unit_len)
        t = decode(t, final_len)
    elif route == "streaming":
        t_pre = 0.0                                      # prefill stream
        t = 0.0                                          # reasoning stream
        pre_done = []
        for u in range(U):
            t_pre = max(t_pre, arrive[u]) + prefill_s(u, 1)
            pre_done.append(t_pre)
        for u in range(U):
            t = max(t, pre_done[u])                      # Algorithm 1: wait for the unit's prefill only
            if first is None and rsn_unit_len[u] > 0:
                ttft = sum(src_unit_len[: u + 1])
            t = decode(t, rsn_unit_len[u])
        if first is None:
            ttft = sum(src_unit_len)
        t = max(t, pre_done[-1] if pre_done else 0.0)
        t = decode(t, final_len)
    else:
        raise ValueError("route must be batch, interleaved or streaming")
    return RouteTimeline(route, int(ttft), float(first if first is not None else t), float(input_end), float(t),
                         float(t - input_end))
