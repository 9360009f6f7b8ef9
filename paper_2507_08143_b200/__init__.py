"""B200-native implementation of Compactor's prefill-time KV-cache compression pass.

The product is the C-ABI library built from `csrc/` (see `include/compactor.h`); `binding`
is a thin ctypes wrapper over it and `inputs` makes the seeded synthetic workloads."""
