"""Streaming episode (instruction prefill + 100 frame steps on a growing cache): the GPU chain
against the oracle, all rows at the sampled steps, and the whole appended cache at the end."""
import numpy as np
import pytest
import torch

from oracle import step_oracle as so
from paper_2512_10310_b200 import binding as B
from paper_2512_10310_b200 import workloads as W
from tests.helpers import GpuStep, bf16_ulp_distance, check_output, f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("layer", [0, 13, 27])
def test_streaming_episode_sampled_steps(layer):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = W.STREAM_7B
    handle = B.evlnCreate(0)
    try:
        T = cfg.final_len
        gs = GpuStep(handle, "bf16", cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, T, cfg.rope_theta,
                     cfg.instruction_len)
        kc = np.zeros((T, cfg.num_kv_heads, cfg.head_dim))
        vc = np.zeros_like(kc)
        sampled = {0, 1, 25, 50, 100}
        for s in range(cfg.num_steps + 1):
            L, n = cfg.call(s)
            x = W.make_new_tokens(cfg.step_config(s, layer))
            g = gs.step(L, x["q_new"], x["k_new"], x["v_new"])
            if s in sampled:
                # the oracle's step rotates, rounds and appends the new keys itself and attends all rows
                r = so.step(f64(x["q_new"]), f64(x["k_new"]), f64(x["v_new"]), kc, vc, L, cfg.rope_theta, storage="bf16")
                check_output("bf16", g["out"], g["lse"], r["out"], r["lse"])
            else:
                # oracle cache only: rotate + round the new keys, copy the values
                kc[L:L + n] = so.round_bf16(so.rope(f64(x["k_new"]), L, cfg.rope_theta))
                vc[L:L + n] = f64(x["v_new"])
        assert L + n == T
        assert bf16_ulp_distance(gs.k_cache.permute(1, 0, 2), kc).max() <= 1
        assert np.array_equal(f64(gs.v_cache.permute(1, 0, 2)), vc)
    finally:
        B.evlnDestroy(handle)
