"""B200-native SwiLA recurrence: C-ABI CUDA library + thin Python binding.

``workloads`` (seeded synthetic inputs) is importable anywhere; ``binding`` loads the
compiled CUDA library and raises if it is missing -- there is no CPU fallback."""
