// The library is built as ONE translation unit: the kernels share a device status word and inline
// PTX helpers, and nothing needs relocatable device code.
#include "internal.cuh"
#include "ptx.cuh"

#include "pack.cu"
#include "pack_nvfp4.cu"
#include "actq.cu"
#include "gemm_i8.cu"
#include "gemm_i8_fewrows.cu"
#include "gemm_i8_midrows.cu"
#include "gemm_fp4.cu"
#include "gemm_fp4_pair.cu"
#include "glue.cu"
#include "api.cu"
#include "static_ws.cu"
