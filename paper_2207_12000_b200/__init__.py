"""gnnpre: block-wise multi-hop feature aggregation on one B200 (CUDA library + thin binding).

`from paper_2207_12000_b200 import binding` loads lib/libgnnpre.so, which
`paper_2207_12000_b200.build.build()` compiles with nvcc for sm_100a.
"""
from . import build  # noqa: F401
