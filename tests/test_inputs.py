"""The seeded input generators: bf16 rounding, determinism, frequency ranking (Section 2.1)."""
import numpy as np
import torch

from paper_2603_05210_b200 import inputs


def test_bf16_rounding_matches_torch_round_to_nearest_even():
    rng = np.random.default_rng(0)
    a = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 0.02,
                        rng.standard_normal(20000).astype(np.float32) * 50,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40], dtype=np.float32)])
    ours = inputs.f32_to_bf16_bits(a)
    ref = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    back = inputs.bf16_bits_to_f32(ours)
    assert np.array_equal(back, torch.from_numpy(a).to(torch.bfloat16).float().numpy())


def test_normal_bf16_is_seeded_and_thread_count_independent():
    a = inputs.normal_bf16((3, (1 << 22) + 5), 0.02, seed=9, threads=1)
    b = inputs.normal_bf16((3, (1 << 22) + 5), 0.02, seed=9, threads=4)
    c = inputs.normal_bf16((3, (1 << 22) + 5), 0.02, seed=10, threads=4)
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    f = inputs.bf16_bits_to_f32(a[0, :200000])
    assert abs(f.std() - 0.02) < 2e-4 and abs(f.mean()) < 2e-4


def test_hidden_state_row_scale_range():
    h = inputs.bf16_bits_to_f32(inputs.hidden_states_bf16(64, 4096, seed=3, row_scale=(0.5, 2.0))).reshape(64, 4096)
    s = h.std(axis=1)
    assert s.min() > 0.45 and s.max() < 2.1 and s.max() / s.min() > 1.5


def test_frequency_ranking_orders_by_count_then_id():
    tok = np.array([5, 5, 2, 9, 9, 2, 7, 5], dtype=np.int32)
    order, cnt = inputs.frequency_ranking(tok, 12)
    assert list(order[:4]) == [5, 2, 9, 7] and list(cnt[:5]) == [3, 2, 2, 1, 0]
    assert list(order[4:]) == [0, 1, 3, 4, 6, 8, 10, 11]
    assert sorted(order.tolist()) == list(range(12))


def test_zipf_stream_is_seeded_and_head_heavy():
    a = inputs.zipf_token_stream(1000, 1.1, 50000, seed=1)
    assert np.array_equal(a, inputs.zipf_token_stream(1000, 1.1, 50000, seed=1))
    assert a.dtype == np.int32 and a.min() >= 0 and a.max() < 1000
    _, cnt = inputs.frequency_ranking(a, 1000)
    assert cnt[0] > 5 * cnt[20] > 0


def test_smallest_prefix_exact_integer_threshold():
    cnt = np.array([50, 30, 15, 4, 1, 0, 0])
    assert inputs.smallest_prefix_with_coverage(cnt, 19, 20) == 3      # 95/100 exactly meets >=
    assert inputs.smallest_prefix_with_coverage(cnt, 96, 100) == 4
    assert inputs.smallest_prefix_with_coverage(cnt, 1, 1) == 5
    assert inputs.smallest_prefix_with_coverage(cnt, 1, 100) == 1


def test_make_case_shapes():
    c = inputs.make_case("t", d=64, V_trim=100, M=3, k=2, seed=5, V_full=1000, n_tokens=5000, keep_stream=True)
    assert c.W_full.shape == (1000, 64) and c.h.shape == (3, 64) and c.keep_ids.shape == (100,)
    assert np.array_equal(c.keep_ids, c.d2t) and len(set(c.keep_ids.tolist())) == 100
    c95 = inputs.make_case("t", d=64, V_trim=None, M=1, k=1, seed=5, V_full=1000, n_tokens=5000,
                           coverage_target=(19, 20), keep_stream=True)
    assert 1 <= c95.V_trim < 1000
