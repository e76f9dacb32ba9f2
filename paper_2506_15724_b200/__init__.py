"""B200-native MadaKV prefill-to-decode KV-cache eviction pass (C-ABI CUDA library + thin Python binding)."""
__all__ = ["binding", "synth"]
