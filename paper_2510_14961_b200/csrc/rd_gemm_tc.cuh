// placeholder interface (tensor-core GEMM arrives in the next step)
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include "../../include/rd.h"
namespace rd {
struct TcWeight { CUtensorMap map; bool valid = false; int n_out = 0, K = 0; };
struct TcAct { CUtensorMap map; bool valid = false; int rows = 0, K = 0; };
static inline int tc_init_driver() { return RD_E_STATE; }
static inline int tc_make_weight(TcWeight*, const void*, int, int) { return RD_E_STATE; }
static inline int tc_make_act(TcAct*, const void*, int, int) { return RD_E_STATE; }
static inline size_t tc_partial_elems(size_t, const rd_config&) { return 0; }
static inline int tc_gemm(cudaStream_t, const TcAct&, const TcWeight&, int, int, float*, size_t, const float*, int,
                          float*, size_t, int*, uint64_t*) { return RD_E_INVALID_ARG; }
}
