"""PolarQuant (arXiv 2502.02617) KV-cache encode / decode-attention hot path for B200 (sm_100a).

`api` binds the C ABI of include/polarquant.h; `synthetic` draws seeded inputs.  Importing the
package does not load the CUDA library; the first API call does, and raises if it was not built.
"""
from . import synthetic  # noqa: F401
from .api import *  # noqa: F401,F403
from .api import GeneralConfig, GeneralPolarQuantCache, PagedPolarQuantCache, Paging, PolarQuantCache, PolarQuantError  # noqa: F401
from .sharding import gather_partials, shard_positions  # noqa: F401
