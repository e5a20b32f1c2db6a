"""The seeded generators: determinism, shapes, and the planted-repeat structure."""
import numpy as np

from sdv_inputs import CONFIGS, bf16_bits_to_f32, f32_to_bf16_bits, get_config, make_context, make_weights


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -2.5, 0.0], dtype=np.float32)
    b = bf16_bits_to_f32(f32_to_bf16_bits(x))
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: goes to the even mantissa (1.0);
    # 1 + 3*2^-8 is a tie between 1 + 2^-7 and 1 + 2^-6: goes to 1 + 2^-6.
    assert b.tolist() == [1.0, 1.0, 1.0 + 2 ** -7, 1.0 + 2 ** -6, -2.5, 0.0]


def test_weights_deterministic_and_thread_independent():
    cfg = get_config("mini_gqa")
    a = make_weights(cfg, threads=1)
    b = make_weights(cfg, threads=5)
    assert np.array_equal(a.emb, b.emb)
    assert np.array_equal(a.layers[2].wd, b.layers[2].wd)
    assert a.lm_head is None and a.layers[0].bq is not None
    c = make_weights(cfg, seed=1)
    assert not np.array_equal(a.emb, c.emb)
    assert a.layers[0].wq.shape == (cfg.n_q_heads * cfg.head_dim, cfg.d_model)
    assert a.layers[0].wd.shape == (cfg.d_model, cfg.d_ffn)


def test_context_has_planted_repeats():
    cfg = get_config("tiny")
    ctx = make_context(cfg)
    assert ctx.shape == (512,) and ctx.dtype == np.int32
    assert ctx.min() >= 0 and ctx.max() < cfg.vocab
    spans = ctx.reshape(-1, cfg.span)
    copies = sum(any(np.array_equal(spans[t], spans[s]) for s in range(t)) for t in range(1, len(spans)))
    assert copies >= 8            # exactly 8 were planted; chance collisions of 16 tokens do not happen
    assert np.array_equal(ctx, make_context(cfg))
    assert not np.array_equal(ctx, make_context(cfg, seed=1))


def test_zipf_head_is_heavy():
    cfg = get_config("qwen1.5b")
    ctx = make_context(cfg)
    _, counts = np.unique(ctx, return_counts=True)
    # Zipf(1.1) over 151936 ranks puts ~9% of the mass on rank 1 and ~35% on the top 16
    assert counts.max() / len(ctx) > 0.05
    assert np.sort(counts)[-16:].sum() / len(ctx) > 0.25


def test_all_configs_meet_layout_constraints():
    for cfg in CONFIGS.values():
        assert cfg.d_model % 64 == 0 and cfg.d_ffn % 64 == 0 and cfg.vocab % 16 == 0
        assert cfg.head_dim in (64, 128) and cfg.n_q_heads % cfg.n_kv_heads == 0
