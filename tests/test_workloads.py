"""The seeded input generators: reproducible, device-independent, shaped like the configs."""
import numpy as np
import torch

from paper_2602_15318_b200 import workloads as W


def test_tensor_stream_matches_host_stream():
    key = W.stream_key(42, 3)
    t = W.splitmix64_tensor(key, 1000, 64, "cpu")
    assert [int(x) & W._M64 for x in t] == [W.splitmix64((key + i) & W._M64) for i in range(1000, 1064)]


def test_normal_table_statistics_and_determinism():
    a = W.normal_bf16(7, 1, (1 << 18,), "cpu", chunk=1 << 16)
    b = W.normal_bf16(7, 1, (1 << 18,), "cpu", chunk=1 << 18)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))      # chunking changes nothing
    f = a.float()
    assert abs(f.mean()) < 0.01 and abs(f.std() - 1) < 0.01 and f.abs().max() < 4.5
    c = W.normal_bf16(7, 2, (1 << 18,), "cpu")
    assert not torch.equal(a.view(torch.int16), c.view(torch.int16))


def test_config_shapes():
    c1 = W.make_config(0)
    assert c1.q.shape == (1, 8, 28, 128) and c1.k.shape == (1, 4, 2056, 128)
    assert c1.parents.tolist() == [[-1, 0, 1, 2, 3, 4, 5, 6]]
    assert c1.kv_bytes() == 2056 * 2048
    par = W.random_tree_parents(W.config_seed(2), 4, 64)
    assert par[0] == -1 and all(-1 <= p < i for i, p in enumerate(par))
    lens = W.ragged_lengths(W.config_seed(4), 5, 8)
    assert all(8192 <= n <= 32768 for n in lens)
    idx = W.c4_anchor_list(8)
    assert len(idx) == 456 and idx[0] == 25664 and idx[-1] == 26119


def test_heavy_rows_shift_keys():
    plain = W.make_verify_case(3, [512], 4, "chain")
    heavy = W.make_verify_case(3, [512], 4, "chain", heavy_frac=0.05, n_visual=[400])
    diff = (plain.k.float() - heavy.k.float()).abs().amax(dim=3)[0]    # [4, cap]
    for h in range(4):
        rows = torch.nonzero(diff[h] > 0).flatten()
        assert len(rows) == 20 and int(rows.max()) < 400
    assert torch.equal(plain.v.view(torch.int16), heavy.v.view(torch.int16))
