"""B200-native LU-KV prefill KV-cache compression path (score -> allocate -> select -> gather).

The compute lives in ``liblukv.so`` (hand-written CUDA for sm_100a behind a C ABI, see
``include/lukv.h``); :mod:`paper_2602_08585_b200.lukv` is the thin binding and
:mod:`paper_2602_08585_b200.synth` draws the seeded synthetic workloads.
"""
__all__ = ["lukv", "synth"]
