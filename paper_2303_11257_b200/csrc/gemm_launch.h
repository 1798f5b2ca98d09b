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

// Batch description of one launch: nb0 x nb1 problems; element strides of each matrix between
// consecutive problems of the outer (index 0) and inner (index 1) batch dimension.
struct BatchDesc {
  int64_t nb0 = 1, nb1 = 1;
  int64_t a[2] = {0, 0}, b[2] = {0, 0}, out[2] = {0, 0};
  bool batched() const { return nb0 * nb1 > 1; }
};

// Builds the tensor maps, picks the tile configuration and launches the kernel for
// ES-byte operands (1 = FP8, 2 = BF16 / F16) with the given operand layouts and epilogue kind.
template <int ES, bool A_MN, bool B_MN>
us_status launch_gemm(const us_mat* A, const us_mat* B, GemmParams& p, const EpiMats& em, int epi, const BatchDesc& bd,
                      cudaStream_t stream);

}  // namespace us
