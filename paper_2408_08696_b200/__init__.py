"""Token Recycling verify-and-recycle step for one B200: hand-written sm_100a
kernels behind a C-ABI library, with a thin ctypes binding (`binding`) and the
seeded synthetic workloads (`synth`)."""
