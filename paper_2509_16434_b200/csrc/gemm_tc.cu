// placeholder: tensor-core GEMMs (forwarding to the CUDA-core kernels until they land)
#include "gemm.cuh"
int tc_gemm_fwd(const ConvGeom &g, const bf16 *X, const bf16 *W, const FwdEpilogue &e, int32_t *, cudaStream_t st) {
    return simt_gemm_fwd(g, X, W, e, st);
}
int tc_gemm_dgrad(const ConvGeom &, const bf16 *, int, const bf16 *, int, const DgradEpilogue &, int32_t *,
                  cudaStream_t) {
    return PPO_ERR_UNSUPPORTED;
}
int tc_gemm_wgrad(const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *X, float *dW, int32_t *, cudaStream_t st) {
    return simt_gemm_wgrad(g, dY, ldy, X, dW, st);
}
