"""Small, self-contained invocations for kernel profilers (one kernel class each, a few launches).

    python profile_case.py matmul MODE M N K [--simt]    # one dense product, run twice
    python profile_case.py iterate WORKLOAD N_NODES ITERS [--no-graph]  # a (reduced) workload
"""

import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

from paper_2105_09837_b200 import binding as B      # noqa: E402
from paper_2105_09837_b200 import synth             # noqa: E402


def main(argv):
    if argv and argv[0] == "matmul":
        mode, M, N, K = (int(x) for x in argv[1:5])
        flags = B.FLAG_SIMT_GEMM if "--simt" in argv else 0
        rng = np.random.default_rng(0)
        a = rng.standard_normal((K, M) if mode == 2 else (M, K), dtype=np.float32)
        b = rng.standard_normal((N, K) if mode == 0 else (K, N), dtype=np.float32)
        for _ in range(2):
            c, ss = B.matmul(mode, a, b, flags)
        print("sum of squares", ss)
        return 0
    if argv and argv[0] == "iterate":
        w = synth.small(argv[1], int(argv[2]))
        ctx = B.from_inputs(synth.make_inputs(w), flags=B.FLAG_NO_GRAPH if "--no-graph" in argv else 0)
        ctx.step(int(argv[3]))
        print("objective", ctx.objective()[5])
        ctx.destroy()
        return 0
    print(__doc__)
    return 2


if __name__ == "__main__":
    sys.exit(main(sys.argv[1:]))
