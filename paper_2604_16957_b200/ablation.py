"""K-versus-V precision ablation on synthetic data (Sec. 5 of the paper reports, on real activations,
cosine 0.998 for int4 K with full-precision V and 0.994 for full-precision K with int4 V).

    python -m paper_2604_16957_b200.ablation [--context S] [--seed N]

Runs tq_sdpa_mixed_precision_attend four times on the same seeded inputs -- K and V each either the int4
cache or the unquantised fp16 values -- and prints, per variant, the mean and minimum over heads of the
cosine similarity between its output and the all-fp16 output.  Inputs: the Llama-shaped generator of the
parity tests -- plain N(0,1); with four K channels x10 per KV head; and the latter with peaked attention
(q scaled x4), where few tokens dominate the softmax.  Needs a CUDA device.
"""
import argparse
import json

import numpy as np
import torch

from . import inputs as I
from . import tq


def cosines(a, b):
    a, b = a.double(), b.double()
    return ((a * b).sum(-1) / (a.norm(dim=-1) * b.norm(dim=-1))).flatten()


def run(context, seed, q_gain, outliers):
    sh = I.Shape("llama", 1, 64, 8, 128, 128 ** -0.5, k_outlier_channels=outliers)
    k, v = I.make_kv(sh, context, seed)
    q = (I.make_q(sh, seed).astype(np.float32) * q_gain).astype(np.float16)
    kd, vd, qd = (torch.from_numpy(np.ascontiguousarray(x)).cuda() for x in (k, v, q))
    cache = tq.KVCache(sh.B, sh.H_kv, context, sh.d)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tq.tq_kv_quantize_append(cache, kd, vd, status)
    outs = {}
    for name, kk, vv in (("fp16 K, fp16 V", kd, vd), ("int4 K, fp16 V", None, vd), ("fp16 K, int4 V", kd, None),
                         ("int4 K, int4 V", None, None)):
        o, m, l = tq.alloc_partials(sh.B, sh.H_q, sh.d, 8)
        out = torch.empty((sh.B, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
        tq.tq_sdpa_mixed_precision_attend(cache, kk, vv, qd, sh.alpha, 8, o, m, l, status)
        tq.tq_sdpa_int4_combine(o, m, l, out)
        outs[name] = out
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = outs["fp16 K, fp16 V"]
    for name, out in outs.items():
        c = cosines(out, ref)
        print(json.dumps({"context": context, "k_outlier_channels": outliers, "q_gain": q_gain, "variant": name, "cosine_mean": round(float(c.mean()), 5),
                          "cosine_min": round(float(c.min()), 5)}), flush=True)


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--context", type=int, default=8192)
    ap.add_argument("--seed", type=int, default=11)
    args = ap.parse_args()
    assert torch.cuda.is_available(), "needs a CUDA device (there is no CPU path)"
    for outliers, gain in ((0, 1.0), (4, 1.0), (4, 4.0)):
        run(args.context, args.seed, gain, outliers)


if __name__ == "__main__":
    main()
