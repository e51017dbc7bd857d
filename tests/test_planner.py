"""Host-side memory / time model of Section 3.4.3 (no GPU, no extension)."""
import dataclasses
import itertools

import numpy as np
import pytest

from paper_2605_25655_b200 import planner as P
from paper_2605_25655_b200 import synth


def test_parameter_counts_match_the_published_llama2_sizes():
    # the parameter counts of the Llama-2 checkpoints are public: 6,738,415,616 / 13,015,864,320 / 68,976,648,192
    assert P.model_param_count(synth.LLAMA_7B) == 6_738_415_616
    assert P.model_param_count(synth.LLAMA_13B) == 13_015_864_320
    assert P.model_param_count(synth.LLAMA_70B) == 68_976_648_192


def test_memory_formulas_worked_examples():
    s = synth.LLAMA_7B
    # KV = B * S_max * 2 * D_size * D_emb * L / TP
    assert P.kv_bytes_per_device(s, 16, 640) == 16 * 640 * 2 * 2 * 4096 * 32
    assert P.kv_bytes_per_device(s, 16, 640, tp=4) == 16 * 640 * 2 * 2 * 4096 * 32 / 4
    # grouped-query attention stores n_kv_heads * head_dim per key row (70B: 1024, not 8192)
    assert P.kv_bytes_per_device(synth.LLAMA_70B, 1, 1) == 2 * 2 * 1024 * 80
    # Params = Model_size / (TP * PP)
    assert P.params_bytes_per_device(s, tp=2, pp=4) == 6_738_415_616 * 2 / 8
    # the paper's 20 GB clusters: the FP16 7B model alone (13.5 GB) fits one cluster, the 13B one does not
    assert P.fits(P.params_bytes_per_device(synth.LLAMA_7B), 0, 0, 20e9)
    assert not P.fits(P.params_bytes_per_device(synth.LLAMA_13B), 0, 0, 20e9)
    assert P.fits(P.params_bytes_per_device(synth.LLAMA_13B, pp=2), 0, 0, 20e9)
    # strict inequality
    assert not P.fits(10, 5, 5, 20) and P.fits(10, 5, 4, 20)


def test_tp_traffic_and_layer_time():
    # Comm_TP = B * 2 * D_emb * D_size * (TP - 1)
    assert P.comm_tp_bytes(16, 4096, 4) == 16 * 2 * 4096 * 2 * 3
    assert P.comm_tp_bytes(16, 4096, 1) == 0
    # T_clu: TP = 1 is the single-device sum; TP divides attention and FFN and adds two reductions and launches
    assert P.layer_time_tp(1.0, 10.0, 20.0) == 32.0
    assert P.layer_time_tp(1.0, 10.0, 20.0, tp=2, t_all_reduce=0.5, t_launch_group=0.25) == 2 + 15 + 1 + 0.5
    # TP pays off only when the saved compute exceeds the added overhead
    assert P.layer_time_tp(1, 10, 20, tp=2, t_all_reduce=8, t_launch_group=0) > P.layer_time_tp(1, 10, 20)


def test_dp_search_equals_brute_force():
    rng = np.random.default_rng(0)
    for _ in range(50):
        t_p, t_d = rng.uniform(0.1, 50), rng.uniform(0.1, 10)
        pp_p, tp_d, pp_d, b_p = (int(v) for v in rng.integers(1, 6, 4))
        dp, cost = P.search_dp_p(t_p, t_d, pp_p, tp_d, pp_d, b_p, range(1, 33))
        brute = min(((dp2 * pp_p + tp_d * pp_d + b_p) * max(t_p / dp2, t_d), dp2) for dp2 in range(1, 33))
        assert cost == pytest.approx(brute[0]) and dp == brute[1]
    # once prefill is no longer the bottleneck, more prefill replicas only add devices
    dp, _ = P.search_dp_p(t_p=8.0, t_d=4.0, pp_p=1, tp_d=1, pp_d=1, b_p=1)
    assert dp == 2
    assert P.pool_devices(3, 2, 4, 5, 6) == 3 * 2 + 4 * 5 + 6


@pytest.mark.parametrize("shape", [synth.LLAMA_7B, synth.LLAMA_13B, synth.LLAMA_70B])
def test_single_device_plan_respects_the_budget(shape):
    plan = P.plan_single_device(shape, s_max=640, prompt=512)
    assert plan is not None and 1 <= plan.max_batch <= 64 and plan.buf_slots >= 2
    used = plan.params_bytes + plan.buf_slots * plan.kv_bytes_per_slot + plan.scratch_bytes + 2 * 10**9
    assert used < P.B200_HBM_BYTES
    # one more slot would not fit (or the batch is already the library's maximum and slots were maximised)
    assert used + plan.kv_bytes_per_slot >= P.B200_HBM_BYTES
    # a smaller budget never yields a larger plan
    small = P.plan_single_device(shape, s_max=640, prompt=512, budget_bytes=int(0.85 * P.B200_HBM_BYTES))
    if small is not None:
        assert (small.max_batch, small.buf_slots) <= (plan.max_batch, plan.buf_slots)
    assert plan.decode_tokens_per_s == pytest.approx(plan.max_batch / plan.decode_step_s)


def test_plan_reports_when_nothing_fits():
    assert P.plan_single_device(synth.LLAMA_70B, s_max=640, prompt=512, budget_bytes=80 * 10**9) is None


def test_roofline_estimates_are_the_byte_and_flop_counts():
    s = synth.LLAMA_7B_LAYER
    w = P.layer_param_count(s) * 2
    t = P.decode_step_seconds(s, 16, 577, hbm_gbs=1000.0, efficiency=1.0)
    assert t == pytest.approx((w + 16 * 577 * 2 * 2 * 4096) / 1e12)
    f = P.prefill_seconds(s, 16, 512, tflops=1000.0, efficiency=1.0)
    gemm = 2 * 16 * 512 * (P.layer_param_count(s) - 2 * 4096)
    assert f == pytest.approx((gemm + 2 * 16 * 32 * 512 * 512 * 128) / 1e15)


def test_cli_prints_a_plan(capsys):
    assert P.main(["--model", "7b", "--mem-gb", "180"]) == 0
    out = capsys.readouterr().out
    assert '"max_batch": 64' in out
