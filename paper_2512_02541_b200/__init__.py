"""B200-native subsampled global attention (AVGGT, Sec. 4.3): Python binding of libavggt."""

from .binding import (  # noqa: F401
    AVGGT_FLAG_KEEP_FIRST_FRAME, AVGGT_MEAN_FILL, AVGGT_MEAN_OFF, AVGGT_MEAN_UNIT, AvggtError, AvggtParams,
    avggt_build_kv, avggt_build_kv_indexed, avggt_build_kv_noalloc, avggt_build_kv_shard, avggt_shard_assemble, avggt_project_build_kv, avggt_project_workspace_bytes, avggt_check_status, avggt_frame_attn, avggt_global_attn, avggt_global_attn_indexed, avggt_global_attn_shard, avggt_kv_count, avggt_version, avggt_workspace_bytes,
    make_params,
)
from .layer import SubsampledGlobalAttention  # noqa: F401
