"""B200-native reduce + AdamW hot path of SlideDP's synchronous step.

``paper_2609_34162_b200.slidedp`` is the thin binding over the C-ABI CUDA library
(it fails loudly when the library is missing; there is no CPU fallback) and
``paper_2609_34162_b200.workloads`` holds the seeded synthetic inputs. Nothing is
loaded at package import time.
"""
