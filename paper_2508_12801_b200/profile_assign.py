"""Run the assignment solver alone on a synthetic score matrix (for ncu captures of its kernels).

    python -m paper_2508_12801_b200.profile_assign [T] [E] [k] [reps]
"""
import sys

import torch

from . import binding as ms
from . import synth


def main():
    T = int(sys.argv[1]) if len(sys.argv) > 1 else 65536
    E = int(sys.argv[2]) if len(sys.argv) > 2 else 128
    k = int(sys.argv[3]) if len(sys.argv) > 3 else 8
    reps = int(sys.argv[4]) if len(sys.argv) > 4 else 3
    dev = "cuda:0"
    ctx = ms.create(ms.make_params(T, 64, E, k, 1.0), dev)
    logits = synth.logits_like(T, E, 0).to(dev)
    scores = torch.empty_like(logits)
    ms.softtopk_fwd(ctx, logits, scores)
    idx = torch.empty(T, k, dtype=torch.int32, device=dev)
    load = torch.empty(E, dtype=torch.int32, device=dev)
    stats = ms.new_stats(dev)
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ms.assign(ctx, scores, idx, load, stats)
        e1.record()
        torch.cuda.synchronize()
        st = ms.read_stats(stats)
        print(f"assign T={T} E={E} k={k}: {e0.elapsed_time(e1):.3f} ms status={st.status} sweeps={st.sweeps} "
              f"aug={st.augmentations} rounds={st.rounds} cand={st.candidates}")
        base = (ctx.workspace.data_ptr() + 255) // 256 * 256 - ctx.workspace.data_ptr()
        tr = ctx.workspace[base:base + 512].cpu().numpy().view("int32")
        print("  exact-phase kilo-cycles (rebuild, path search, moves), path-search rounds, of the last round run:", tr[44:48].tolist(), "queue entries:", int(tr[41]), "first rebuild kc:", int(tr[42]), "moves split (find token, patch, recompute) kc and arcs moved:", tr[34:38].tolist())
        print("  rows scanned in full per sweep:", tr[64:64 + st.sweeps].tolist())


if __name__ == "__main__":
    main()
