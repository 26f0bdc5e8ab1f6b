"""B200 (sm_100a) library for the hot path of the Hotline heterogeneous embedding pipeline.

``binding`` mirrors the C boundary (include/hotline.h) one to one; ``pipeline.Hotline`` owns the buffers and
issues the calls of one mini-batch in pipeline order.  Importing the package loads libhotline.so and fails
loudly if it has not been built (``python paper_2204_05436_b200/csrc/build.py``); there is no CPU fallback.
"""
from . import binding  # noqa: F401  (loads the shared library)
from .binding import *  # noqa: F401,F403
from .pipeline import Hotline, NativePipelinedHotline, PipelinedHotline  # noqa: F401
