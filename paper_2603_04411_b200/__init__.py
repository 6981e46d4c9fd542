"""libtwkv: token-wise adaptive low-rank KV-cache compression (compress + decode attention) on B200.

  paper_2603_04411_b200.binding    ctypes binding of the C ABI declared in include/twkv.h
  paper_2603_04411_b200.build      builds libtwkv.so in-tree with nvcc (sm_100a)
  paper_2603_04411_b200.workloads  seeded synthetic inputs
  paper_2603_04411_b200.replicas   barrier / max-over-ranks / whole-job rate for runs on several GPUs (replicas, no data-path collective)

The CUDA library is the only implementation: importing `binding` without a built
libtwkv.so raises.
"""
__all__ = ["binding", "build", "workloads", "replicas"]
