"""B200 (sm_100a) fused attention forward, and GEMM + row sum: CUDA kernels behind a C ABI, plus this thin binding."""
from .binding import (AttnError, AttnVariantDesc, attn_fwd, attn_fwd_host, host_workspace_bytes, launch_count, make_desc,  # noqa: F401
                      raw_attn_fwd, status_string, variant_kwargs, version, clear_cache, cache_hits, selftest_timeout)
from .binding import (GemmRowsumDesc, gemm_rowsum, gemm_rowsum_host, gemm_rowsum_host_workspace_bytes,  # noqa: F401
                      gemm_rowsum_launch_count, raw_gemm_rowsum)
