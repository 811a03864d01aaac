"""B200 (sm_100a) gradient compression for data attribution: GraSS / FactGraSS
(arXiv 2505.18976) as hand-written CUDA kernels behind a C ABI.

``binding`` wraps the shared library declared in ``include/grass.h``;
``workloads`` draws the seeded synthetic inputs; ``build`` compiles the library.
"""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    GrassError, GroupedLayers, SjltSpec, FactgrassLayer, factgrass_compress, factgrass_compress_grouped,
    factgrass_compress_grouped_static, FACTGRASS_STATIC_MAX_LAYERS,
    factgrass_compress_varlen, factgrass_compress_grouped_varlen, grass_fim, grass_fim_factor, grass_fim_apply, grass_mask, factmask_compress, factmask_compress_grouped,
    factgrass_grouped_workspace_bytes, grass_compress, grass_random_mask_host, grass_score, grass_sjlt_table,
    grass_validate_mask, mask_to_device, lib, grass_to_bf16, grass_score_bf16, grass_set_tuning, tuning,
)
