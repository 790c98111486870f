// Second level of the column-sum reduction behind Eq. 4's mean token.  Kernels that produce one chunk
// partial per CTA (the stand-alone column-sum kernel and the restore kernel, which sums the rows it has
// just updated) call fold_group_partials at their end: the last CTA of each group of chunks to arrive
// adds that group's chunk partials in chunk order, so the result does not depend on which CTA was last.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "internal.h"

namespace fv {

// Called by ALL threads of the CTA after they have stored their part of chunk partial (b, chunk).
// Returns true, with the group partial written, if this CTA was the last of its group.
__device__ __forceinline__ bool fold_group_partials(int b, int chunk, int nchunks, int group, int ngroups, int C4,
                                                    const float4* __restrict__ chunk_partial,
                                                    float4* __restrict__ group_partial, unsigned int* tickets) {
  __shared__ int s_last;
  const int g = chunk / group;
  __threadfence();  // this thread's partial is visible device-wide before the ticket is taken
  __syncthreads();
  if (threadIdx.x == 0) {
    const int first = g * group;
    const int members = min(group, nchunks - first);
    unsigned int* t = tickets + (size_t)b * kMaxGroups + g;
    const unsigned int prev = atomicAdd(t, 1u);
    s_last = (prev == (unsigned int)(members - 1));
    if (s_last) *t = 0u;  // every member has arrived: leave the counter ready for the next launch
  }
  __syncthreads();
  if (!s_last) return false;
  __threadfence();
  const int first = g * group;
  const int last = min(nchunks, first + group);
  const float4* src = chunk_partial + (size_t)b * nchunks * C4;
  for (int c4 = threadIdx.x; c4 < C4; c4 += blockDim.x) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    int c = first;
    for (; c + 8 <= last; c += 8) {
      float4 v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = __ldcg(src + (size_t)(c + i) * C4 + c4);
#pragma unroll
      for (int i = 0; i < 8; ++i) { acc.x += v[i].x; acc.y += v[i].y; acc.z += v[i].z; acc.w += v[i].w; }
    }
    for (; c < last; ++c) {
      const float4 v = __ldcg(src + (size_t)c * C4 + c4);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    group_partial[((size_t)b * ngroups + g) * C4 + c4] = acc;
  }
  return true;
}

}  // namespace fv
