"""CPU tests of the arrival-process timeline (no GPU, no library): closed forms on constant call durations."""
import pytest

from paper_2510_17238_b200 import arrival


def test_three_routes_closed_forms():
    n, m, f = [10, 10, 10], [4, 4, 4], 2
    rate = 10.0                                   # tokens per second: a unit arrives every second
    P, D = 0.05, 0.1                              # every prefill call 50 ms, every decode step 100 ms
    runs = {r: arrival.simulate(r, n, m, f, lambda u, k: P, lambda r_: D, tokens_per_second=rate)
            for r in ("batch", "interleaved", "streaming")}
    b, i, s = runs["batch"], runs["interleaved"], runs["streaming"]
    assert b.input_end_s == i.input_end_s == s.input_end_s == pytest.approx(3.0)
    # batch: everything after the input: prefill, 14 decode steps
    assert b.ttft_tokens == 30 and b.first_token_s == pytest.approx(3.0 + P + D)
    assert b.delay_s == pytest.approx(P + 14 * D)
    # interleaved and streaming start after the first unit
    assert i.ttft_tokens == s.ttft_tokens == 10
    assert i.first_token_s == s.first_token_s == pytest.approx(1.0 + P + D)
    # reasoning about a unit (0.4 s) is shorter than the gap between units (1 s): both are input-bound here, and the
    # last unit's reasoning plus the final stage is what is left after the input ends
    assert s.delay_s == pytest.approx(P + 4 * D + 2 * D)
    assert i.delay_s == pytest.approx(P + 4 * D + 2 * D)


def test_streaming_hides_prefill_when_reasoning_is_the_bottleneck():
    n, m, f = [10] * 4, [20] * 4, 0
    rate = 100.0                                  # a unit every 0.1 s; reasoning about it takes 2 s
    P, D = 0.5, 0.1
    i = arrival.simulate("interleaved", n, m, f, lambda u, k: P, lambda r_: D, tokens_per_second=rate)
    s = arrival.simulate("streaming", n, m, f, lambda u, k: P, lambda r_: D, tokens_per_second=rate)
    # interleaved pays every prefill on the critical path, streaming only the first one
    assert i.done_s == pytest.approx(0.1 + 4 * P + 80 * D)
    assert s.done_s == pytest.approx(0.1 + P + 80 * D)
    assert s.delay_s < i.delay_s
    with pytest.raises(ValueError):
        arrival.simulate("other", n, m, f, lambda u, k: P, lambda r_: D)


def test_call_durations_may_depend_on_the_call():
    n, m, f = [5, 5], [1, 1], 1
    s = arrival.simulate("streaming", n, m, f, lambda u, k: 0.01 * (u + 1), lambda r: 0.1 * (r + 1), tokens_per_second=5.0)
    # unit 1 arrives at 1 s, prefilled at 1.01; token 0 at 1.11; unit 2 arrives at 2 s, prefilled at 2.02; token 1 at 2.22;
    # final token (0.3 s) at 2.52
    assert s.first_token_s == pytest.approx(1.11) and s.done_s == pytest.approx(2.52)
    b = arrival.simulate("batch", n, m, f, lambda u, k: 0.01 * k, lambda r: 0.1 * (r + 1), tokens_per_second=5.0)
    assert b.first_token_s == pytest.approx(2.0 + 0.02 + 0.1) and b.ttft_tokens == 10
