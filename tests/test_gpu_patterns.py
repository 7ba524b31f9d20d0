"""Every delivery pattern, produced by the device's own hash path.

At p = 0.5 all 2^(W K) receive patterns of a bucket of K packets are equally likely. The GPU runs enough
steps that every pattern turns up, the steps are grouped by the recv_bits the device reports, and for every
pattern the estimate must equal the masked sum over the received count written out here. The same for the
2^((W-1) K) broadcast patterns against stale_bits: the replicas that took the broadcast hold the new wire
value, the others their old packet.
"""
import numpy as np
import pytest
import torch

import paper_2507_07114_b200 as L

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("W,K,flags", [(4, 1, 0), (3, 2, 0), (2, 2, L.LOSSY_REGISTER_PATH), (4, 1, L.LOSSY_REGISTER_PATH)])
def test_all_receive_and_stale_patterns_are_observed_and_each_equals_the_enumeration(W, K, flags):
    P = 1024                      # one bulk-copy tile per packet (or four register-kernel chunks)
    n = K * P
    steps = 24 * 2 ** (W * K)
    ctx = L.lossy_init(W=W, n=n, packet_elems=P, p_grad=0.5, p_param=0.5, seed=12345, grad_dtype=torch.float32,
                       replica_dtype=torch.float32, optimizer="sgd", lr=1.0, flags=flags)
    rng = np.random.default_rng(3)
    g_np = rng.standard_normal((W, n)).astype(np.float32)
    grads = [torch.from_numpy(g_np[i]).cuda() for i in range(W)]
    master = torch.zeros(n, device="cuda")
    reps = [torch.zeros(n, device="cuda") for _ in range(W)]
    ghat = torch.zeros(n, device="cuda")
    recv = torch.zeros(K, dtype=torch.int64, device="cuda")
    stale = torch.zeros(K, dtype=torch.int64, device="cuda")
    count = torch.zeros(K, dtype=torch.uint8, device="cuda")
    seen_recv, seen_stale = set(), set()
    pps = (K + W - 1) // W
    for t in range(1, steps + 1):
        before = [r.clone() for r in reps]
        L.lossy_fused_step(ctx, t, grads, master, None, None, reps, ghat, count, recv, stale)
        torch.cuda.synchronize()
        r_bits, s_bits = recv.cpu().numpy().view(np.uint64), stale.cpu().numpy().view(np.uint64)
        gh, th = ghat.cpu().numpy(), master.cpu().numpy()
        seen_recv.add(tuple(int(x) for x in r_bits))
        seen_stale.add(tuple(int(x) for x in s_bits))
        for k in range(K):
            sl = slice(k * P, (k + 1) * P)
            who = [i for i in range(W) if (int(r_bits[k]) >> i) & 1]
            assert int(count[k]) == len(who)
            want = np.zeros(P, np.float32)
            for i in who:                           # ascending worker order, fp32
                want = want + g_np[i, sl]
            if who:
                want = want / np.float32(len(who))
            assert np.array_equal(gh[sl], want), f"step {t} packet {k} pattern {who}"
            owner = k // pps
            assert not (int(s_bits[k]) >> owner) & 1
            for i in range(W):
                got = reps[i][sl].cpu().numpy()
                if (int(s_bits[k]) >> i) & 1:
                    assert np.array_equal(got, before[i][sl].cpu().numpy())     # kept its old packet
                else:
                    assert np.array_equal(got, th[sl])                          # took the new value
    L.lossy_destroy(ctx)
    assert len(seen_recv) == 2 ** (W * K), f"{len(seen_recv)} of {2 ** (W * K)} receive patterns seen"
    # per packet the owner never misses: (W-1) free bits per packet
    assert len(seen_stale) == 2 ** ((W - 1) * K), f"{len(seen_stale)} of {2 ** ((W - 1) * K)} stale patterns seen"
