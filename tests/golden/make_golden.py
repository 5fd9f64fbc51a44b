"""Writes tests/golden/tiny_fp32_round.json: the float64 checker's result on the
tiny fp32 workload (a regression anchor for the checker itself; the paper
prints no worked numeric example for this path).  Calls only oracle/ and the
seeded input generator.   Usage: python tests/golden/make_golden.py"""
import json
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import csd_oracle as orc                    # noqa: E402
from paper_2411_11925_b200 import inputs as gen         # noqa: E402

out = orc.round_from_inputs(gen.make_round_inputs(gen.WORKLOADS["tiny_fp32"]))
doc = {
    "source": "oracle/csd_oracle.py round_from_inputs on workload tiny_fp32 (Alg. 1, Eq. 8, Cor. 1)",
    "x0": out["x0"].tolist(), "mu1_p": out["mu1_p"].tolist(),
    "logratio": out["logratio"].tolist(), "n_accept": [int(v) for v in out["n_accept"]],
    "n_prop": [int(v) for v in out["n_prop"]], "x_new": out["x_new"].tolist(),
}
with open(os.path.join(HERE, "tiny_fp32_round.json"), "w") as f:
    json.dump(doc, f, indent=1)
print("logratio", out["logratio"], "n_accept", out["n_accept"], "n_prop", out["n_prop"])
