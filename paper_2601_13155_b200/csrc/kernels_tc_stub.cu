// placeholder until the tcgen05 kernels land
#include "spts_common.cuh"
namespace spts {
spts_status tc_init(spts_ctx*) { return SPTS_OK; }
int tc_sumsq_parts(int n_out) { return n_out / 128; }
spts_status launch_tc_gemm(spts_ctx*, int, const TcGemmArgs&) { return SPTS_ERR_UNSUPPORTED; }
spts_status launch_tc_attention(spts_ctx*, const bf16*, const bf16*, const bf16*, int, int, bf16*) { return SPTS_ERR_UNSUPPORTED; }
}
