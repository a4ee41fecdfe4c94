"""B200-native parameter-server hot path: W logical workers' CNN gradient step and
the server-side reduce / apply / replay of the gradient queue (sm_100a CUDA behind a
C ABI).  `ps` is the thin ctypes binding; `synth` the seeded input generators."""

__all__ = ["ps", "synth"]
