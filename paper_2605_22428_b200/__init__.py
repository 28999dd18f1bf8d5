"""MultiWrite dispatch / AllGather pack-and-deliver for B200 (sm_100a).

`workloads` holds the seeded input generators; `binding` is the ctypes front end of
the CUDA library (libmw.so).  The library is loaded on first use and a missing or
unloadable library is an error: there is no CPU fallback.
"""
