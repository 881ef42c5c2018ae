"""The seeded generators: pinned against a big-integer restatement, checked for slice
consistency and for the first two moments."""
import torch

from workloads import configs, gen


def test_mix64_matches_bigint():
    idx = torch.tensor([0, 1, 2, 12345678901, (1 << 62) + 17], dtype=torch.int64)
    got = gen.hash_u64(7, gen.TID_X, idx)
    key = gen.stream_key(7, gen.TID_X)
    for i, g in zip(idx.tolist(), got.tolist()):
        want = gen.mix64_py(i * 0x9E3779B97F4A7C15 + key)
        assert (g & ((1 << 64) - 1)) == want


def test_slices_are_consistent_and_streams_differ():
    full = gen.normal_f32(3, gen.TID_W_DOWN, 0, 5000, 0.5)
    part = gen.normal_f32(3, gen.TID_W_DOWN, 1234, 1000, 0.5, chunk=333)
    assert torch.equal(full[1234:2234], part)
    other = gen.normal_f32(3, gen.TID_W_GATE_UP, 0, 5000, 0.5)
    assert not torch.equal(full, other)
    assert not torch.equal(full, gen.normal_f32(4, gen.TID_W_DOWN, 0, 5000, 0.5))


def test_moments():
    v = gen.normal_f32(0, gen.TID_X, 0, 1 << 20, 2.0).double()
    assert abs(v.mean().item()) < 0.01
    assert abs(v.std().item() - 2.0) < 0.01
    kurt = ((v - v.mean()) ** 4).mean() / v.var() ** 2 - 3.0
    assert abs(kurt.item() + 0.15) < 0.03  # Irwin-Hall n=8


def test_slab_equals_full_tensor_slice():
    cfg = configs.small_variant(configs.CONFIGS[1], T=8, d=64, F=32, E=4)
    full = configs.make_w_gate_up(cfg)
    assert torch.equal(full[3], configs.w_gate_up_slab(cfg, 3))
    assert torch.equal(configs.make_w_down(cfg)[5], configs.w_down_slab(cfg, 5))  # shared expert slab


def test_zipf_config_has_dead_experts():
    cfg = configs.small_variant(configs.CONFIGS[3], T=2048, d=128, F=64)
    x = configs.make_x(cfg)
    logits = configs.make_logits(cfg, x)
    top = torch.topk(logits, cfg.k, dim=1).indices
    counts = torch.bincount(top.flatten(), minlength=cfg.E)
    assert (counts == 0).sum().item() >= cfg.n_dead
    assert counts.max().item() > 4 * counts.float().mean().item()  # skewed
