"""B200-native SNLP (Structured Newton Layer Parallelism) hot path.

``paper_2605_17842_b200.snlp``  -- thin binding over the C-ABI CUDA library (loads it on import and
                                    fails loudly if it is missing).
``paper_2605_17842_b200.synth`` -- seeded synthetic inputs (no arithmetic of the method).
"""
