// Single translation unit of libsinglequant: the device status word and the kernels share
// file-scope device symbols, so everything is compiled together (no relocatable device code).
#include "sq_gemm.cu"
#include "sq_gemm_pair.cu"
#include "sq_gemm_decode.cu"
#include "sq_gemv.cu"
#include "sq_rotate_quant.cu"
#include "sq_rotate_quant_tc.cu"
#include "sq_rotate_quant_st.cu"
#include "sq_rotate_quant_pair.cu"
#include "sq_linear_fused.cu"
#include "sq_rotation_host.cu"
#include "sq_api.cu"
#include "sq_noalloc.cu"
