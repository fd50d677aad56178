"""B200-native PolluxSched optimizer core: speedup tables, population fitness and the
genetic-algorithm step as CUDA kernels behind a C-ABI library.

`paper_2008_12260_b200.synth` draws seeded synthetic inputs; `paper_2008_12260_b200.api`
is the thin binding over `libpolluxsched.so` (imported lazily so that input generation
works on machines without the compiled library; every compute call requires it).
"""

__all__ = ["synth"]
