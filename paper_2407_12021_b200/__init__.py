"""B200-native verification step of adaptive draft-verification decoding (ADED).

`inputs` holds the seeded synthetic workload generators; `binding` wraps the C-ABI
shared library built from `csrc/` (see include/aded.h).
"""
