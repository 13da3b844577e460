"""The seeded input generators: batched and per-request forms give the same elements."""
import torch

from paper_2512_09427_b200 import workloads as wl


def test_batched_kv_rows_equal_the_per_request_ones():
    runs = [(3, 0, 4), (9, 5, 5), (4, 2, 9), (1 << 33, 100, 103)]
    for dtype in (torch.bfloat16, torch.float32):
        a = wl.kv_rows_batch(7, 1, [r for r, _, _ in runs], wl.KIND_V, [x for _, x, _ in runs],
                             [y for _, _, y in runs], 2, 16, dtype)
        b = torch.cat([wl.kv_rows(7, 1, r, wl.KIND_V, x, y, 2, 16, dtype) for r, x, y in runs])
        assert a.shape == (14, 2, 16) and torch.equal(a, b)


def test_streams_differ_by_key_and_are_standard_normal():
    x = wl.gen_normal((1, 2, 3), 0, 1 << 16, torch.float32)
    y = wl.gen_normal((1, 2, 4), 0, 1 << 16, torch.float32)
    assert not torch.equal(x, y)
    assert abs(float(x.mean())) < 0.02 and abs(float(x.std()) - 1.0) < 0.02
    assert torch.equal(wl.gen_normal((1, 2, 3), 100, 50, torch.float32), x[100:150])
