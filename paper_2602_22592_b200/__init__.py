"""B200-native pQuant decoupled linear layer (1-bit branch + routed high-precision
experts under feature scaling): hand-written sm_100a CUDA kernels behind a C ABI.

`paper_2602_22592_b200.binding` exposes the C entry points under their own
names; `paper_2602_22592_b200.inputs` generates the seeded synthetic workloads.
Nothing is loaded at import time; the shared library is opened on first use and
its absence is an error, never a fallback.
"""
