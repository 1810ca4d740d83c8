"""B200 (sm_100a) implementation of Fathom's decode-step hot path behind a C ABI (include/fathom.h).

`binding` loads libfathom.so (built in-tree by `build.py`) and raises if it is missing.
"""
