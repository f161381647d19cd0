"""DENSE sampling + GraphSage forward + DistMult on one B200: Python binding of libmgdense."""
from . import inputs  # noqa: F401
from .api import (BACKING_HBM, BACKING_HOST, CORRUPT_BOTH, CORRUPT_DST, CORRUPT_SRC, GEMM_FP32,  # noqa: F401
                  GEMM_TF32, Context, Dense, GatModel, LpBatch, MgError, Model, comet_autotune, comet_bias, comet_plan,
                  load_library)
