"""Writes tests/golden/cfg1_oracle.json from the CPU oracle alone (configuration 1:
512x512 INT4 g=128, grid init, 10 rounds, seed 0).  Run: python tests/golden/make_golden.py"""
import json
import os
import sys
import zlib

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2605_08692_b200 import synth  # noqa: E402  (input generator only)

c = synth.config1()
r = oracle.fit_layer(c["W"], c["mode"], c["group"], c["rounds"], X=c["X"], init="grid")
out = dict(T=[float(v) for v in r["T"].ravel()], trace=[float(v) for v in r["trace"]],
           T_bf16=[int(v) for v in r["T_bf16"].ravel()], sigma_ones=int(r["sigma"].sum()),
           E_final=float(r["E_final"]), codes_crc32=zlib.crc32(r["codes"].tobytes()))
json.dump(out, open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg1_oracle.json"), "w"), indent=1)
print("wrote cfg1_oracle.json")
