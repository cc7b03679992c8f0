// The static block pattern (paper Section 3.1) at block granularity.
#pragma once
#include <cuda_runtime.h>

namespace lg {

struct PatternDev {
  int nB;       // ceil(L / block)
  int mode;     // 0 full causal, 1 sink+window, 2 strided+local
  int ns, nw;   // sink blocks, window blocks (own block included; one more when the window is token-exact)
  int stride, nl;
  // Optional pruning by packed documents (device code only; null on the host and for plain patterns):
  // doc_start[i] of the one sequence the lists are built for, and the block size in tokens.
  const int* doc_start;
  int block;
};

// Block (qb, kb) holds at least one allowed (query, key) pair.  Causality needs kb <= qb
// (the diagonal block always contains the pair i == j); the rest of the predicate only
// depends on the block indices (Section 3.1 patterns).
__host__ __device__ __forceinline__ bool block_active(const PatternDev& p, int qb, int kb) {
  if (kb > qb) return false;
#ifdef __CUDA_ARCH__
  // The first row of a query block belongs to the earliest document of the block, so it sees the most:
  // a key block that ends before that document starts holds nothing any row of the block may see.
  // (A superset of the blocks that are really needed; what is left over is masked in the kernels.)
  if (p.doc_start && (kb + 1) * p.block <= p.doc_start[qb * p.block]) return false;
#endif
  if (p.mode == 0) return true;
  if (p.mode == 1) return kb < p.ns || qb - kb < p.nw;
  return qb - kb < p.nl || kb % p.stride == 0;
}

}  // namespace lg
