"""Host-side checks of the synthetic workload generator (shapes, seeding, structure)."""
import numpy as np
import torch

from paper_2604_16734_b200.workloads import CONFIGS, Workload, reduced


def test_chunk_schedules_match_the_configs():
    c = {k: [n for _, n in v.chunks()] for k, v in CONFIGS.items()}
    assert c["C1"] == [64] * 9 + [32]
    assert c["C2"] == [128] * 4 + [64, 64]
    assert c["C3"] == [576] * 5 + [128]
    assert c["C4"] == [196] * 64 + [128]
    assert c["C5"] == [1024] * 36 + [256]
    assert c["T4"] == [784] * 10 + [128]
    assert [n for _, n in CONFIGS["T4"].scaled(chunk=512).chunks()] == [512] * 15 + [160, 128]
    for cfg in CONFIGS.values():
        sched = cfg.chunks()
        assert sched[0][0] == 0 and sum(n for _, n in sched) == cfg.n_tokens
        assert all(sched[i + 1][0] == sched[i][0] + sched[i][1] for i in range(len(sched) - 1))
    assert [CONFIGS[k].n_tokens for k in ("C1", "C2", "C3", "C4", "C5")] == [608, 640, 3008, 12672, 37120]


def test_shapes_dtype_seeding():
    cfg = CONFIGS["C1"]
    q, k, v = Workload(cfg).layer(0)
    assert q.shape == (608, 4, 64) and k.shape == (608, 1, 64) and v.shape == k.shape
    assert q.dtype == torch.float32
    q2, _, _ = Workload(cfg).layer(0)
    assert torch.equal(q, q2)
    q3, _, _ = Workload(cfg, seed=1).layer(0)
    assert not torch.equal(q, q3)
    cfg = reduced(CONFIGS["C4"], n_layers=2, n_units=3)
    wl = Workload(cfg)
    qa, ka, _ = wl.layer(0)
    qb, kb, _ = wl.layer(1)
    assert qa.dtype == torch.bfloat16 and qa.shape == (3 * 196 + 128, 32, 128) and ka.shape[1] == 8
    assert not torch.equal(ka, kb)
    assert torch.isfinite(qa.float()).all()


def test_vision_tokens_are_spatially_and_temporally_redundant():
    cfg = reduced(CONFIGS["C4"], n_units=4).scaled(mix_layers=False)
    _, k, _ = Workload(cfg).layer(0)
    x = k[: cfg.n_vision].float().reshape(4, 14, 14, -1)
    def corr(a, b):
        a = a.flatten(); b = b.flatten()
        return float(np.corrcoef(a.numpy(), b.numpy())[0, 1])
    assert corr(x[:, :, :-1], x[:, :, 1:]) > 0.6          # neighbouring patches
    assert corr(x[:-1], x[1:]) > 0.6                      # consecutive frames (rho = 0.9, noise 0.3)
    text = k[cfg.n_vision:].float()
    assert abs(corr(text[:-1], text[1:])) < 0.1           # text tokens are white


def test_hybrid_schedule_covers_the_prefix_once():
    for cfg in CONFIGS.values():
        sched = cfg.chunks_hybrid()
        assert sched[0] == (0, min(cfg.budget, cfg.n_vision))
        pos = 0
        for p, n in sched:
            assert p == pos and 1 <= n and (n <= cfg.chunk or p == 0)
            pos += n
        assert pos == cfg.n_tokens
        # vision and text never share a block
        assert all(not (p < cfg.n_vision < p + n) for p, n in sched)
