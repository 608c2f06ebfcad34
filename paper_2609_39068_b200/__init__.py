"""B200-native sparse decode attention (Quest page selection + split-K paged attention +
H2O statistic) behind a C ABI.  ``binding`` is the thin ctypes layer over
``libsparse_engine.so``; ``workloads`` builds seeded synthetic inputs."""

__all__ = ["binding", "workloads"]
