"""Pins for the oracle's characterisation statistics (Section 3, Figures 2-4): dense restatement on toy traces,
closed forms on the MLP chain, conservation identities on the DNN-shaped configs."""
import numpy as np

import helpers
from paper_2310_09443_b200 import traces


def test_toys_against_dense(oracle):
    rng = np.random.default_rng(5150)
    for trial in range(200):
        K = int(rng.integers(1, 16)); N = int(rng.integers(1, 9))
        tr = traces.random_toy(rng, K, N, max_bytes=5000, max_ns=100000)
        used = helpers.dense_matrix(tr)
        uses, first, last, periods = helpers.brute_vitality(tr)
        start = helpers.brute_start(tr)
        v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
        c = oracle.characterize(tr.K, v, tr.tensor_bytes, np.asarray(start), tr.host_bw, tr.ssd_bw)
        exp_active = [sum(int(tr.tensor_bytes[i]) for i in range(N) if used[k][i]) for k in range(K)]
        assert c.active_bytes.tolist() == exp_active
        assert c.summary.tolist() == [max(exp_active), exp_active.index(max(exp_active))]
        lh = [0] * 64; sl = np.zeros((41, 45), np.int64); hide = [0, 0]
        for (i, u, w) in periods:
            L = start[w] - start[u + 1]; s = int(tr.tensor_bytes[i])
            lh[L.bit_length() - 1] += 1
            sl[min(s.bit_length() - 1, 40), min(L.bit_length() - 1, 44)] += 1
            for X, bw in ((0, tr.ssd_bw), (1, tr.host_bw)):
                if 2 * (-((-s * 10 ** 9) // bw)) <= L:
                    hide[X] += 1
        assert c.len_hist.tolist() == lh and np.array_equal(c.size_len_hist, sl) and c.hide.tolist() == hide


def test_mlp_chain_and_conservation(oracle):
    tr = traces.config0_mlp_chain()
    v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    start = oracle.slot_clock(tr.kernel_ns)
    c = oracle.characterize(tr.K, v, tr.tensor_bytes, start, tr.host_bw, tr.ssd_bw)
    # fwd_l uses W_l, A_{l-1}, A_l: kernel l-1
    for l in (1, 7, 32):
        assert c.active_bytes[l - 1] == tr.tensor_bytes[66 + l - 1] + tr.tensor_bytes[l - 1] + tr.tensor_bytes[l]
    assert c.len_hist.sum() == 93 == c.size_len_hist.sum()
    for cfg in (1, 2):
        tr = traces.make_config(cfg)
        v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
        start, P0, peak, slot = oracle.timeline(tr)
        c = oracle.characterize(tr.K, v, tr.tensor_bytes, start, tr.host_bw, tr.ssd_bw)
        # every distinct (kernel, tensor) incidence contributes the tensor's size exactly once
        assert int(c.active_bytes.astype(object).sum()) == int((tr.tensor_bytes.astype(object) * v.num_uses.astype(object)).sum())
        assert np.all(c.active_bytes <= P0)                       # what a kernel uses is alive while it runs
        assert c.len_hist.sum() == len(v.period_tensor) and np.all(c.hide <= len(v.period_tensor)) and c.hide[1] >= c.hide[0]
        g = oracle.geometry(start, tr.tensor_bytes, v.period_tensor, v.period_prev_use, v.period_next_use, tr.host_bw, tr.ssd_bw)
        L = start[v.period_next_use] - start[v.period_prev_use + 1]
        assert c.hide[0] == int((2 * g.transfer_ns[0] <= L).sum()) and c.hide[1] == int((2 * g.transfer_ns[1] <= L).sum())
