"""PTQTP dual-trit-plane decode linear layer for NVIDIA B200 (sm_100a).

The product is the C-ABI library ``libptqtp.so`` (sources under ``csrc/``, declarations in
``include/ptqtp.h``); ``binding`` marshals torch tensors into its calls and ``inputs`` holds
the seeded synthetic workloads.  Nothing here computes on the CPU: if the CUDA library is
missing the binding raises.
"""
__all__ = ["binding", "inputs"]
