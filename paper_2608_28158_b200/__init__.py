"""Tree-packed chunkwise linear attention for B200 (sm_100a).

Thin Python binding over the C-ABI library ``libharts_la.so`` (declared in
``include/harts_la.h``).  Every step of the path runs in the library's CUDA kernels or its
host planner; PyTorch only owns device memory and streams.  There is no CPU fallback: if the
library cannot be loaded the import of :mod:`paper_2608_28158_b200.binding` fails.
"""
from .binding import (  # noqa: F401
    HARTS_BF16, HARTS_FP32, HARTS_FLAG_FMA_KERNELS, HARTS_FLAG_CHECK_TABLES, HARTS_FLAG_ROUND_LAUNCHES, HartsError, Plan, Workspace, harts_la_bwd, harts_la_bwd_finish, harts_la_bwd_static, harts_la_selftest_timeout,
    harts_la_bwd_seqs, harts_la_check, harts_la_fwd, harts_la_fwd_seqs, harts_la_plan, harts_la_strerror,
    harts_la_workspace_bytes, lib, run_fwd_bwd, run_fwd_bwd_host, harts_la_step_host, HostPipeline, expand_trajectories, harts_la_expand, harts_la_gk_workspace_bytes, harts_la_gk_fwd, harts_la_gk_bwd,
)
from .logp import (  # noqa: F401
    harts_logp_positions, harts_logp_csr, harts_logp_multiplicity, harts_logp_fwd, harts_logp_bwd, harts_logp_fwd_shard, harts_logp_combine,
)
from .conv import harts_conv_index, harts_conv_fwd, harts_conv_scratch_bytes, harts_conv_bwd  # noqa: F401
from .attn import AttnIndex, harts_attn_index, harts_attn_fwd, harts_attn_bwd  # noqa: F401
from .mb import MbPlan, harts_mb_plan  # noqa: F401
