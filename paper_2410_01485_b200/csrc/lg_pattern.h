// The static block pattern (paper Section 3.1) at block granularity.
#pragma once
#include <cuda_runtime.h>

namespace lg {

struct PatternDev {
  int nB;       // ceil(L / block)
  int mode;     // 0 full causal, 1 sink+window, 2 strided+local
  int ns, nw;   // sink blocks, window blocks (own block included; one more when the window is token-exact)
  int stride, nl;
};

// Block (qb, kb) holds at least one allowed (query, key) pair.  Causality needs kb <= qb
// (the diagonal block always contains the pair i == j); the rest of the predicate only
// depends on the block indices (Section 3.1 patterns).
__host__ __device__ __forceinline__ bool block_active(const PatternDev& p, int qb, int kb) {
  if (kb > qb) return false;
  if (p.mode == 0) return true;
  if (p.mode == 1) return kb < p.ns || qb - kb < p.nw;
  return qb - kb < p.nl || kb % p.stride == 0;
}

}  // namespace lg
