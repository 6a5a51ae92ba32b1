"""Helper of test_gpu_prefill_forms.py: Thinformer Express prefill of the listed shapes with the library as the
environment configures it; outputs and coresets go to the .npz file named on the command line."""
import sys

import numpy as np
import torch

# log2_nout, mbar, rounds R, head dim, batch, query heads, KV heads
SHAPES = [
    (6, 4, 3, 64, 2, 4, 2),       # d = 64, two batch entries, level-0 calls of 16 points
    (7, 5, 3, 128, 1, 8, 2),      # grouped queries
    (8, 2, 3, 128, 1, 4, 4),      # Subsample in Express round r = 2 (one token kept of 4)
    (6, 0, 3, 128, 1, 2, 1),      # mbar = 0: no Halve call inside a segment
    (6, 1, 4, 64, 1, 4, 2),       # strata of 32 tokens in Express round r = 3
    (6, 0, 6, 64, 1, 2, 1),       # strata of 1024 tokens: a pair of query tiles lies inside one stratum
    (7, 3, 4, 128, 2, 2, 2),
]


def run(path):
    import paper_2606_10944_b200 as elm
    from paper_2606_10944_b200.workloads import WORKLOADS, generate
    out = {}
    for i, (ln, mbar, R, d, B, Hq, Hkv) in enumerate(SHAPES):
        n = (1 << ln) * 4 ** R
        wl = WORKLOADS["cfg5"].scaled(batch=B, q_heads=Hq, kv_heads=Hkv, n=n, n_q=n, d=d)
        Q, K, V = generate(wl, seed=5, want_q=True)
        before = elm.launch_count()
        O, idx, _ = elm.express_prefill(Q.cuda(), K.cuda(), V.cuda(), ln, mbar, seed=3, precision="fp32")
        torch.cuda.synchronize()
        out[f"O{i}"] = O.float().cpu().numpy()
        out[f"idx{i}"] = idx.cpu().numpy()
        out[f"launches{i}"] = np.int64(elm.launch_count() - before)
    np.savez(path, **out)


if __name__ == "__main__":
    run(sys.argv[1])
