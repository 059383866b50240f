// Second kernel of the fused row reduction (included by the C-ABI file only).
#pragma once

#include "cg_kernel.cuh"

namespace cg {

// Second pass of the fused row reduction: one thread per row combines its row's partials in slot order.
__global__ void row_finalize_kernel(const float* __restrict__ ws, float* __restrict__ out, long long rows, int slots, int op) {
  const long long row = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (row >= rows) return;
  if (op == REDUCE_LOGSUMEXP) {
    const float2* w = reinterpret_cast<const float2*>(ws) + row * slots;
    float mx = -INFINITY;
    for (int s = 0; s < slots; ++s) mx = fmaxf(mx, w[s].x);
    float sum = 0.0f;
    for (int s = 0; s < slots; ++s)
      if (w[s].x > -INFINITY) sum += w[s].y * expf(w[s].x - mx);
    out[row] = mx + logf(sum);
  } else {
    const float* w = ws + row * slots;
    float acc = op == REDUCE_SUM ? 0.0f : -INFINITY;
    for (int s = 0; s < slots; ++s) acc = op == REDUCE_SUM ? acc + w[s] : fmaxf(acc, w[s]);
    out[row] = acc;
  }
}

}  // namespace cg
