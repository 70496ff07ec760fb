"""The seeded input generator: deterministic, block-addressable, and shaped as the workload recipes say."""
import numpy as np

from paper_2412_16187_b200 import workloads as wl


def test_blocks_are_addressable_and_deterministic():
    w = wl.CONFIGS["llama3_8b_gqa"].scaled(prompt_len=64, budget=16, decode_steps=8)
    full = wl.gen_tokens(w, "k", 0, 3, 0, 72)
    assert np.array_equal(full, wl.gen_tokens(w, "k", 0, 3, 0, 72))
    assert np.array_equal(full[1:3, :, 10:20], wl.gen_tokens(w, "k", 1, 2, 10, 10))
    q = wl.gen_tokens(w, "q", 0, 1, 0, 4)
    assert q.shape == (1, w.n_kv_heads * w.group_size, 4, w.head_dim)
    dec = wl.gen_decode_inputs(w, "k", 2, 3)  # steps 2..4 are tokens 66..68
    assert np.array_equal(dec[:, :3].transpose(1, 2, 0, 3), full[:, :, 66:69])
    assert not np.array_equal(wl.gen_tokens(w.scaled(seed=9), "k", 0, 1, 0, 8), full[:1, :, :8])


def test_iid_normal_statistics():
    w = wl.CONFIGS["tiny"]
    x = wl.gen_tokens(w, "k", 0, 1, 0, 128).astype(np.float64).ravel()
    n = x.size
    assert abs(x.mean()) < 4 / np.sqrt(n) and abs(x.var() - 1) < 4 * np.sqrt(2 / n)
    assert abs(np.mean(x ** 3)) < 4 * np.sqrt(15 / n) and abs(np.mean(x ** 4) - 3) < 4 * np.sqrt(96 / n)
    W = wl.gen_W(w)
    assert W.shape == (64, 8) and W.dtype == np.float32 and abs(W.std() - 1) < 0.15
    assert not np.array_equal(wl.gen_W(w, layer=1), W)


def test_outlier_channels_and_drift():
    w = wl.CONFIGS["llama2_7b_layer"].scaled(prompt_len=2048, budget=64, decode_steps=0)
    k = wl.as_f64(w, wl.gen_tokens(w, "k", 0, 1, 0, 2048))[0]  # [heads, N, d]
    std = k.std(axis=1)
    for h in range(4):
        big = np.sort(np.argsort(std[h])[-4:])
        assert np.all(std[h][big] > 7) and np.sum(std[h] > 5) == 4  # exactly four channels at ~10x
    assert len({tuple(np.sort(np.argsort(std[h])[-4:])) for h in range(8)}) > 1  # chosen per head
    # slow mean drift: first and last quarter means differ on non-outlier channels, by at most ~|m_c|
    small = std[0] < 5
    drift = k[0][1536:][:, small].mean(axis=0) - k[0][:512][:, small].mean(axis=0)
    assert 0.2 < np.abs(drift).mean() < 2.0


def test_cluster_keys_and_ragged_budgets():
    w = wl.CONFIGS["throughput_batch"]
    b = w.budgets()
    assert b.shape == (64,) and b.min() >= 512 and b.max() <= 4096 and len(set(b.tolist())) > 50
    assert np.array_equal(w.prompt_lens(), 2 * b)
    k = wl.as_f64(w, wl.gen_tokens(w, "k", 0, 1, 0, 1024))[0, 0]  # [N, d]
    std = k.std(axis=0)
    small = np.argsort(std)[:-4]
    # 16 tight clusters: nearest-centre residual (sigma 0.5) is far below the spread of centres (2.0)
    x = k[:, small]
    d2 = ((x[:64, None, :] - x[None, :, :]) ** 2).sum(-1)
    d2[np.arange(64), np.arange(64)] = np.inf
    nearest = d2.min(axis=1)  # distance to the nearest other key: same cluster -> ~2*0.25*d
    assert np.median(nearest) < 0.25 * 2 * small.size * 1.6
    assert x.var(axis=0).mean() > 2.0
