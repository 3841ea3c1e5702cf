// SAP step 2, CSC X: conflict bits of all candidate pairs.  x_a^T x_b of two sparse columns is the
// intersection of two ascending row lists.  One CTA owns candidate a and stages its column in shared
// memory; each warp takes 32 consecutive later candidates b (one per lane), every lane merges its own
// column b against the staged column a, and one ballot yields the 32 conflict bits of that mask word.
// Products are accumulated in row order, so the result does not depend on the launch shape.
#include "strads_internal.cuh"

namespace strads {
namespace {

constexpr int kThreads = 256;
constexpr int kStage = 1024;          // entries of column a staged in shared memory (longer columns: global)

__global__ void __launch_bounds__(kThreads) k_gram_csc(Problem p, const int* __restrict__ cand, int n_cand,
                                                        float* __restrict__ gram_dbg, int only_if_short, int window) {
  chain_begin();
  if (only_if_short && !p.st->window_short) return;
  if (window && p.st->prefer_walk && ((p.st->round / (unsigned)p.part_count) & 63ull) != 0) return;   // the window attempt is being skipped
  __shared__ int arow[kStage];
  __shared__ float aval[kStage];
  const int a = blockIdx.x;
  if (a >= n_cand) return;
  const int ja = cand[a];
  const long long a0 = p.xptr[ja];
  const int na = (int)(p.xptr[ja + 1] - a0);
  const bool staged = na <= kStage;
  if (staged)
    for (int q = threadIdx.x; q < na; q += kThreads) { arow[q] = p.xrow[a0 + q]; aval[q] = p.xv[a0 + q]; }
  __syncthreads();
  const int* ar = staged ? arow : p.xrow + a0;
  const float* av = staged ? aval : p.xv + a0;
  const double n2a = p.n2[ja];
  const double rho = (double)p.rho;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  for (int w = (a >> 5) + warp; w < p.mask_words; w += kThreads / 32) {
    const int b = w * 32 + lane;
    bool hit = false;
    if (b < n_cand && b != a) {
      const int jb = cand[b];
      const float dot = sparse_dot(ar, av, na, p, jb);
      const double den = sqrt(n2a * p.n2[jb]);
      hit = den > 0.0 && fabs((double)dot) >= rho * den;
      if (gram_dbg != nullptr) {
        gram_dbg[(long long)a * n_cand + b] = dot;
        if (b > a) gram_dbg[(long long)b * n_cand + a] = dot;
      }
    } else if (b == a && gram_dbg != nullptr) {
      gram_dbg[(long long)a * n_cand + a] = (float)n2a;
    }
    const unsigned int word = __ballot_sync(0xffffffffu, hit);
    if (lane == 0) p.conflict[(long long)a * p.mask_words + w] = word;
  }
}

}  // namespace

cudaError_t launch_gram_csc(const Problem& p, const int* cand, int n_cand, float* gram_dbg, bool only_if_short,
                            bool window, cudaStream_t s) {
  return launch_chained(k_gram_csc, n_cand, kThreads, 0, s, p, cand, n_cand, gram_dbg, only_if_short ? 1 : 0, window ? 1 : 0);
}

}  // namespace strads
