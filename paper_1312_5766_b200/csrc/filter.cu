// SAP step 2 / Algorithm 1 "choose a set B1 of <= P coefficients from U such that |x_j^T x_k| < rho":
// greedy first-fit over the candidates in sampling order, on the conflict bits of the Gram kernel.
//
// The walk is a serial chain (whether candidate i is kept depends on every earlier decision), and each
// keep needs the conflict row of the kept candidate: a dependent memory access.  To take that latency
// off the chain, one CTA prefetches the rows of the next 32 still-unblocked candidates together into
// shared memory (they are the only ones that can be kept next), and one warp then resolves those 32
// in order against the running `blocked` mask entirely in shared memory.
#include "strads_internal.cuh"

namespace strads {
namespace {

constexpr int kThreads = 256;
constexpr int kBatch = 32;

__global__ void __launch_bounds__(kThreads) k_filter(Problem p, const int* __restrict__ cand, int n_cand,
                                                      int* __restrict__ kept_out) {
  extern __shared__ unsigned int sm[];
  const int W = p.mask_words;
  unsigned int* blocked = sm;                    // [W]
  unsigned int* rows = sm + W;                   // [kBatch][W]
  __shared__ int pos[kBatch];
  __shared__ int s_m, s_cursor, s_kept, s_examined, s_done;
  const int tid = threadIdx.x, lane = tid & 31;
  const bool no_filter = (p.flags & STRADS_FLAG_NO_FILTER) != 0;

  for (int w = tid; w < W; w += kThreads) blocked[w] = 0u;
  if (tid == 0) { s_cursor = 0; s_kept = 0; s_examined = 0; s_done = 0; }
  __syncthreads();

  if (no_filter) {
    const int nk = min(n_cand, p.n_keep);
    for (int i = tid; i < p.n_keep; i += kThreads) kept_out[i] = i < nk ? cand[i] : -1;
    if (tid == 0) { p.st->counts[1] = nk; p.st->counts[2] = nk; p.st->counts[3] = 0; p.st->amb_count = 0; }
    return;
  }

  while (true) {
    // 1. the next <= kBatch candidates that are not blocked yet
    if (tid < 32) {
      int m = 0;
      int cur = s_cursor;
      while (cur < n_cand && m < kBatch) {
        const int wbase = (cur >> 5) + lane;           // 32 mask words at a time
        unsigned int freew = 0u;
        if (wbase < W) {
          freew = ~blocked[wbase];
          const int first = wbase << 5;
          if (first < cur) freew &= (cur - first >= 32) ? 0u : (0xffffffffu << (cur - first));
          if (first + 32 > n_cand) freew &= (n_cand - first <= 0) ? 0u : (0xffffffffu >> (first + 32 - n_cand));
        }
        // lanes in order append their free positions
        for (int l = 0; l < 32 && m < kBatch; ++l) {
          unsigned int fw = __shfl_sync(0xffffffffu, freew, l);
          const int base = ((cur >> 5) + l) << 5;
          while (fw && m < kBatch) {
            const int b = __ffs(fw) - 1;
            fw &= fw - 1;
            if (lane == 0) pos[m] = base + b;
            ++m;
          }
        }
        if (m < kBatch) cur = ((cur >> 5) + 32) << 5;  // all 32 words consumed
      }
      if (lane == 0) s_m = m;
    }
    __syncthreads();
    const int m = s_m;
    if (m == 0) {                                      // list exhausted
      if (tid == 0) s_examined = n_cand;
      break;
    }
    // 2. fetch their conflict rows together
    for (int e = tid; e < m * W; e += kThreads) {
      const int r = e / W, w = e - r * W;
      rows[r * W + w] = __ldcg(&p.conflict[(long long)pos[r] * W + w]);
    }
    __syncthreads();
    // 3. resolve in order
    if (tid < 32) {
      int nk = s_kept;
      int last = -1;
      bool full = false;
      for (int q = 0; q < m; ++q) {
        const int i = pos[q];
        const bool is_blocked = (blocked[i >> 5] >> (i & 31)) & 1u;
        last = i;
        if (!is_blocked) {
          if (lane == 0) kept_out[nk] = cand[i];
          ++nk;
          for (int w = (i >> 5) + lane; w < W; w += 32) blocked[w] |= rows[q * W + w];
          __syncwarp();
          if (nk == p.n_keep) { full = true; break; }
        }
      }
      if (lane == 0) {
        s_kept = nk;
        s_cursor = last + 1;
        if (full) { s_examined = last + 1; s_done = 1; }
      }
    }
    __syncthreads();
    if (s_done) break;
  }
  __syncthreads();
  const int nk = s_kept;
  for (int i = nk + tid; i < p.n_keep; i += kThreads) kept_out[i] = -1;
  if (tid == 0) { p.st->counts[1] = s_examined; p.st->counts[2] = nk; p.st->counts[3] = 0; p.st->amb_count = 0; }
}

}  // namespace

size_t filter_smem_bytes(const Problem& p) { return (size_t)(kBatch + 1) * p.mask_words * sizeof(unsigned int); }

// Kernel-wide attribute: the largest size any handle can need (see prepare_sample).
cudaError_t prepare_filter(const Problem&) {
  return cudaFuncSetAttribute(k_filter, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)((kBatch + 1) * (STRADS_MAX_CANDIDATES / 32) * sizeof(unsigned int)));
}

cudaError_t launch_filter(const Problem& p, const int* cand, int n_cand, int* kept_out, cudaStream_t s) {
  k_filter<<<1, kThreads, filter_smem_bytes(p), s>>>(p, cand, n_cand, kept_out);
  return cudaGetLastError();
}

}  // namespace strads
