"""sonic: fused LLM sampling and speculative verification for one B200 (sm_100a).

The product is the C-ABI library built from csrc/ (declared in include/sonic.h);
`binding` marshals torch tensors into it and `workloads` draws seeded synthetic
inputs.  Nothing in this package falls back to the CPU.
"""
