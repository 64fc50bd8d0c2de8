"""libjackpot: the OBRS token pass of Jackpot (arxiv 2602.06107) on one B200.

The work is done by hand-written sm_100a kernels behind a C ABI
(``include/jackpot.h``); :mod:`.binding` marshals torch tensors into it,
:mod:`.runner` allocates outputs around the calls, :mod:`.inputs` makes the
seeded synthetic workloads.  Importing the package loads nothing; the first
binding call loads ``libjackpot.so`` and raises if it is missing.
"""
__all__ = ["binding", "runner", "inputs", "build", "parallel"]
