"""Writes the stored expected values under tests/golden/.

Calls only the CPU oracle and the seeded input generators; nothing here touches the
CUDA library.  Run from the repository root:  python tests/golden/make_golden.py
"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import stairs_oracle as so  # noqa: E402
from paper_2407_19947_b200 import workloads as wl  # noqa: E402


def main():
    w = wl.workload(1)
    tsrc, _ = wl.make_sources(w)
    tgt = so.OracleModel(w.target, tsrc)
    toks = so.greedy_generate(tgt, wl.prompt_tokens(w), w.max_new)
    with open(os.path.join(HERE, "cfg1_greedy_tokens.txt"), "w") as f:
        f.write("# Stand-alone greedy continuation (32 tokens) of the tiny config's target model,\n"
                "# computed by the CPU oracle (paper Section 3.1, Fig. 2).  The paper prints no\n"
                "# numeric example; this file guards the oracle and the generators against drift.\n")
        f.write(" ".join(str(t) for t in toks) + "\n")
    print(toks)


if __name__ == "__main__":
    main()
