"""Writes paper_2403_00176_b200/cfg5_gate_bias.txt: one gate bias per block of the gated skip
network, chosen so that about 40-70 % of a calibration batch skips each block.

Calls only the oracle and the workload generator.  For block i the target skip fraction is
q_i ~ U(0.4, 0.7) (seeded); with the logits z sorted ascending and m = round(q_i * B), the bias is
b_i = -(z_(m) + z_(m+1)) / 2 so that exactly m samples have z + b_i <= 0.  Decisions of earlier
blocks change the features of later ones, so the pass is repeated a few times from the previous
biases until the skip counts settle.  Usage:  python tests/golden/calibrate_cfg5_gates.py [passes]
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import interp as O  # noqa: E402
from paper_2403_00176_b200 import workloads as WL  # noqa: E402
from paper_2403_00176_b200.workloads import bf16_round  # noqa: E402

OUT = os.path.join(ROOT, "paper_2403_00176_b200", "cfg5_gate_bias.txt")


def main(passes: int = 3):
    wl = WL.cfg5(calibrated=False)
    n_blocks = len([k for k in wl.consts if k.endswith(".gb")])
    B = wl.meta["B"]
    rng = np.random.Generator(np.random.PCG64(WL.SEED0 + 5000 + 998))
    q = rng.uniform(0.4, 0.7, n_blocks)
    req = wl.batch(999)[0]          # calibration batch: a seed the benchmark batches never use
    bias = np.array([float(wl.consts[f"b{i}.gb"][0]) for i in range(n_blocks)])
    if os.path.exists(OUT):      # resume from the last written biases
        prev = [float(ln) for ln in open(OUT) if ln.strip() and not ln.startswith("#")]
        if len(prev) == n_blocks:
            bias = np.array(prev)
    for it in range(passes):
        for i in range(n_blocks):
            wl.consts[f"b{i}.gb"] = bf16_round(np.array([bias[i]], np.float32))
        env = O.run(wl.ir, wl.consts, req.inputs)
        new = bias.copy()
        for i in range(n_blocks):
            z = env[f"logit{i}"].reshape(-1) - float(wl.consts[f"b{i}.gb"][0])   # logits without the bias
            zs = np.sort(z)
            m = int(round(q[i] * B))
            m = min(max(m, 1), B - 1)
            new[i] = -(zs[m - 1] + zs[m]) / 2.0
        skipped = [int((~env[f"gate{i}"].reshape(-1)).sum()) for i in range(n_blocks)]
        print(f"pass {it}: skipped per block {skipped}", flush=True)
        # a block's logits depend only on the decisions of earlier blocks, so each pass settles at
        # least one more block exactly; keep the biases of blocks that already meet their target
        ok = [abs(skipped[i] - int(round(q[i] * B))) <= 1 for i in range(n_blocks)]
        bias = np.where(ok, bias, new)
        if all(ok):
            break
    with open(OUT, "w") as f:
        f.write("# gate bias per block of the default gated skip network (written by tests/golden/calibrate_cfg5_gates.py)\n")
        for b in bias:
            f.write(f"{float(bf16_round(np.array([b], np.float32))[0])!r}\n")
    print("wrote", OUT)


if __name__ == "__main__":
    main(int(sys.argv[1]) if len(sys.argv) > 1 else 3)
