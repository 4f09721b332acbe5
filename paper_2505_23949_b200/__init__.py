"""B200-native TSENOR hot path: transposable N:M mask solver (block loader,
log-domain Dykstra, greedy rounding, local-search repair, bit-packed masks)
as hand-written sm_100a CUDA behind a C ABI, plus a thin ctypes binding."""
__all__ = ["binding", "synth"]
