"""Host-side arithmetic of the benchmark (no GPU): the byte count behind the span-search roofline and the rule
that picks the denominator of the tensor roofline."""
import bench


def test_search_key_bytes_is_the_closed_form_work_count():
    # sum over i < L of floor(sqrt(i+1)): the values the work-count pin of the oracle uses
    for L, want in ((16, 38), (64, 316), (4096, 172768), (65536, 11152256), (262144, 89347840)):
        assert bench.search_key_bytes(1, 1, L, 1, 1) == want
    # one 256-byte row per (position, stride, KV head) in the second configuration
    assert bench.search_key_bytes(1, 8, 65536, 128, 2) == 11152256 * 8 * 256
    # a window of w removes floor(sqrt(w)) strides from every position that has them
    full, win = bench.search_key_bytes(1, 1, 4096, 1, 1), bench.search_key_bytes(1, 1, 4096, 1, 1, window=1088)
    assert win == sum(max(0, int((i + 1) ** 0.5 + 1e-9) - 32) for i in range(4096)) and win < full


def test_tensor_roofline_denominator_rule():
    peaks = {"bf16_tflops": 1600.0, "bf16_tflops_sustained": 1300.0, "_source": "measured"}
    short = bench.tensor_roofline(4e12, 5.0, 0.1, {"sm_mhz": 1200.0, "sm_max_mhz": 1965.0}, peaks)
    assert short["peak"] == 1600.0 and abs(short["achieved"] - 800.0) < 1e-9 and abs(short["frac"] - 0.5) < 1e-12
    full_clock = bench.tensor_roofline(4e12, 5.0, 10.0, {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0}, peaks)
    assert full_clock["peak"] == 1600.0
    long_capped = bench.tensor_roofline(4e12, 5.0, 10.0, {"sm_mhz": 1300.0, "sm_max_mhz": 1965.0}, peaks)
    assert long_capped["peak"] == 1300.0 and abs(long_capped["frac_of_burst"] - 0.5) < 1e-12
    assert abs(long_capped["frac_of_nominal"] - 800.0 / 2250.0) < 1e-12
    assert long_capped["ms_times_sm_mhz"] == 5.0 * 1300.0


def test_both_arms_share_the_config_object():
    from paper_2601_18401_b200 import synth
    c = bench.config_of(synth.CONFIGS[1], 1)
    assert c["workload"] == "prefill_L65536" and c["seq_len"] == 65536 and c["top_k"] == 8 and "model" not in c
