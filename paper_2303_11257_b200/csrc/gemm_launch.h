// Interface between the argument-checking front end (gemm.cu) and the kernel instantiations
// (gemm_inst.cu, compiled once per operand width and layout).
#pragma once
#include <cuda_runtime.h>

#include "../../include/unitscale.h"

namespace us {

struct GemmParams;

// The matrices the epilogue reaches through TMA (aux / skip NULL when unused).
struct EpiMats {
  const us_mat* out;
  const us_mat* aux;
  const us_mat* skip;
};

// Builds the tensor maps, picks the tile configuration and launches the kernel for
// ES-byte operands (1 = FP8, 2 = BF16 / F16) with the given operand layouts and epilogue kind.
template <int ES, bool A_MN, bool B_MN>
us_status launch_gemm(const us_mat* A, const us_mat* B, GemmParams& p, const EpiMats& em, int epi, cudaStream_t stream);

}  // namespace us
