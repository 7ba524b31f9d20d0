"""Host and device evaluate the same delivery indicator as the oracle (bit-exact)."""
import numpy as np
import pytest
import torch

import paper_2507_07114_b200 as L
from oracle import oracle as O

pytestmark = pytest.mark.gpu


def _ctx(p_grad, p_param, seed):
    return L.lossy_init(W=8, n=1024, packet_elems=64, p_grad=p_grad, p_param=p_param, seed=seed,
                        grad_dtype=torch.float32, replica_dtype=torch.float32, optimizer="sgd", lr=0.1)


@pytest.mark.parametrize("seed,p", [(0, 0.1), (12345678901234567, 0.3), (2**64 - 1, 0.01), (7, 0.0)])
def test_device_mask_grid_matches_oracle(seed, p):
    ctx = _ctx(p, min(0.99, p * 2), seed)
    try:
        rng = np.random.default_rng(1)
        steps = [1, 2, 1000, 2**40 + 3]
        for step in steps:
            n = 20000
            src = rng.integers(0, 64, n).astype(np.uint32)
            dst = rng.integers(0, 64, n).astype(np.uint32)
            pk = np.concatenate([np.arange(n // 2, dtype=np.uint64),
                                 rng.integers(0, 2**63, n - n // 2, dtype=np.uint64)])
            for is_param, pp in ((False, p), (True, min(0.99, p * 2))):
                out = torch.zeros(n, dtype=torch.uint8, device="cuda")
                L.lossy_mask_grid(ctx, step, torch.from_numpy(src.astype(np.int32)).cuda(),
                                  torch.from_numpy(dst.astype(np.int32)).cuda(),
                                  torch.from_numpy(pk.view(np.int64)).cuda(), out, is_param)
                got = out.cpu().numpy()
                want = np.array([O.delivered(seed, step, int(s), int(d), int(k), pp)
                                 for s, d, k in zip(src, dst, pk)], dtype=np.uint8)
                assert np.array_equal(got, want)
                host = np.array([L.lossy_mask(ctx, step, int(s), int(d), int(k), is_param)
                                 for s, d, k in zip(src[:2000], dst[:2000], pk[:2000])], dtype=np.uint8)
                assert np.array_equal(host, want[:2000])
        for k in range(200):
            assert L.lossy_hash_u32(seed, 3, k % 5, k % 7, k) == O.hash_u32(seed, 3, k % 5, k % 7, k)
    finally:
        L.lossy_destroy(ctx)
