// The batched GEMM of the MLP producer: argument block shared by the CUDA-core kernels
// (abs_mlp.cu) and the tensor-core kernel (abs_gemm_tc.cu).
#pragma once

#include "abs_internal.cuh"

namespace absk {

// C[z] = epilogue( A[z] * B[z] ), z < batch, fp32 operands with arbitrary strides.
struct GemmArgs {
  const float* A; long long a_rs, a_cs, a_bs;    // element (r, k) at A[z*a_bs + r*a_rs + k*a_cs]
  const float* B; long long b_rs, b_cs, b_bs;    // element (k, c)
  float* C; long long c_rs, c_bs;                // element (r, c) at C[z*c_bs + r*c_rs + c]
  const float* bias; long long bias_bs;          // per column (modes 1, 2)
  const float* mask; long long mask_rs, mask_bs; // shape of C (mode 3)
  int rows, cols, K;
  float alpha;
  int mode;   // 0: alpha*acc   1: relu(acc + bias)   2: acc + bias   3: acc where mask > 0, else 0
};

// Tensor-core route (tcgen05, 3 x TF32 split products, fp32 accumulation in TMEM folded into fp32
// registers every 32 values of k).  Returns false when the shape is not worth a 128 x 128 tile or
// an operand has no contiguous index; the caller then uses the CUDA-core kernels.
// `flag`: device word that receives 1 when a bounded wait ran out (the results are then not valid).
// `drop_loads`: fault injection for tests (no operand tile is ever filled, so every wait runs out).
bool launch_gemm_tc(const GemmArgs& g, int batch, unsigned* flag, long long timeout_cycles, bool drop_loads,
                    cudaStream_t st);

}  // namespace absk
