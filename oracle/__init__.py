"""Adam-mini oracle package -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Plain float64 CPU implementations written from the paper, used only by
tests/, the smoke check and the benchmark's CPU-baseline / reference legs:

  adammini_oracle.c  Algorithm 1 (Adam-mini), one tensor per call, C, float64
  step.py            ctypes loader and the `OracleState` convenience class
  adamw_ref.py       a separately written AdamW (coordinate-wise v) in numpy
  exact.py           exact-rational transcription of Algorithm 1 for tiny cases
  partition_ref.py   Algorithm 2 / Algorithm 3 partition rules in Python

Nothing here imports the CUDA package, and the CUDA package imports nothing
from here.
"""
