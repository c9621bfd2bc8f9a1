// Temporary: entry points not built yet report SF_ERR_UNSUPPORTED.
#include "sf_common.cuh"
extern "C" {
int sf_gemm_workspace_size(int64_t, int64_t, size_t* b) { if (b) *b = 256; return SF_OK; }
int sf_gemm_dense(const void*, int, const void*, int, void*, int64_t, int64_t, int64_t, void*, void*) { return SF_ERR_UNSUPPORTED; }
int sf_gemm_sparse24(const void*, const void*, const void*, void*, int64_t, int64_t, int64_t, void*, void*) { return SF_ERR_UNSUPPORTED; }
int sf_gemm_venom(const void*, const void*, const void*, const void*, void*, int64_t, int64_t, int64_t, int, int, void*, void*) { return SF_ERR_UNSUPPORTED; }
int sf_ffn_workspace_size(const sf_ffn_desc*, size_t*, size_t*) { return SF_ERR_UNSUPPORTED; }
int sf_sparse_ffn_fwd(const sf_ffn_desc*, const void*, const void*, const void*, void*, void*, void*, void*) { return SF_ERR_UNSUPPORTED; }
int sf_sparse_ffn_bwd(const sf_ffn_desc*, const void*, const void*, const void*, const void*, const void*, void*, void*, void*, void*, void*) { return SF_ERR_UNSUPPORTED; }
int sf_dense_ffn_fwd(const sf_ffn_desc*, const void*, const void*, const void*, void*, void*, void*, void*) { return SF_ERR_UNSUPPORTED; }
int sf_dense_ffn_bwd(const sf_ffn_desc*, const void*, const void*, const void*, const void*, const void*, void*, void*, void*, void*, void*) { return SF_ERR_UNSUPPORTED; }
int sf_ctx_view(const sf_ffn_desc*, const void*, int, const void**, size_t*) { return SF_ERR_UNSUPPORTED; }
int sf_ffn_host_staging_size(const sf_ffn_desc*, size_t*) { return SF_ERR_UNSUPPORTED; }
int sf_ffn_step_host(const sf_ffn_desc*, int, const void*, const void*, const void*, const void*, void*, void*, void*, void*, void*, void*, void*, void*) { return SF_ERR_UNSUPPORTED; }
int sf_check_status(void*, void*) { return SF_ERR_UNSUPPORTED; }
}
