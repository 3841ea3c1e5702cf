// Greedy first-fit (SAP step 2 / Algorithm 1 "choose a set B1 ... |x_j^T x_k| < rho") settled from the list of
// conflicting candidate pairs, by one CTA of kNT threads.  Shared by the walk kernel and by the CTA of the
// window Gram kernel that finishes last.
//
// Conflicts are few, so the rule "keep b unless an earlier kept a conflicts with it" is settled in passes over
// the pairs: a candidate with a kept earlier neighbour is out, one whose earlier neighbours are all decided and
// out is kept (a candidate without earlier neighbours at once).  The number of passes is the longest chain of
// such dependencies, two or three in practice; past kSparsePasses the caller falls back on the walk over the
// bit rows.  Stopping at P is a cut of the kept sequence at its P-th member: no decision depends on a later
// position.
#pragma once
#include "strads_internal.cuh"

namespace strads {

constexpr int kSparsePasses = 24;

// Bytes of shared memory the walk needs for n_cand candidates and n_edges listed pairs.
__host__ __device__ inline size_t walk_pairs_smem(int n_cand, unsigned int n_edges) {
  return 3 * (((size_t)n_cand + 15) & ~(size_t)15) + sizeof(unsigned int) * (size_t)n_edges;
}

// Returns whether the walk was settled (uniform over the CTA).  If so, kept_out[0 .. *n_kept) and
// p.kept_pos[0 .. *n_kept) hold the kept coefficients and their positions in the list, and *n_examined the
// position after the P-th kept one (left alone when fewer than P are kept).  n_kept / n_examined: shared memory.
template <int kNT>
__device__ bool walk_from_pair_list(const Problem& p, const int* __restrict__ cand, int n_cand, unsigned int n_edges,
                                    unsigned char* sm, int* __restrict__ kept_out, int* n_kept, int* n_examined) {
  __shared__ int s_scan[kNT / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  unsigned char* state = sm;                                              // 0 undecided, 1 kept, 2 out
  unsigned char* hit = state + ((n_cand + 15) & ~15);                     // has a kept earlier neighbour
  unsigned char* pend = hit + ((n_cand + 15) & ~15);                      // has an undecided earlier neighbour
  unsigned int* e = reinterpret_cast<unsigned int*>(pend + ((n_cand + 15) & ~15));
  for (int i = tid; i < n_cand; i += kNT) { state[i] = 0; hit[i] = 0; pend[i] = 0; }
  for (unsigned int k = tid; k < n_edges; k += kNT) e[k] = __ldcg(p.edges + k);
  __syncthreads();
  bool settled = false;
  for (int pass = 0; pass < kSparsePasses && !settled; ++pass) {
    for (unsigned int k = tid; k < n_edges; k += kNT) {
      const int a = (int)(e[k] >> 16), b = (int)(e[k] & 0xffffu);
      if (state[b] == 0) {
        const unsigned char sa = state[a];
        if (sa == 1) hit[b] = 1;                       // (several threads may store the same value: benign)
        else if (sa == 0) pend[b] = 1;
      }
    }
    __syncthreads();
    int open = 0;
    for (int i = tid; i < n_cand; i += kNT) {
      if (state[i] == 0) {
        if (hit[i]) state[i] = 2;
        else if (!pend[i]) state[i] = 1;
        else open = 1;
        pend[i] = 0;
      }
    }
    settled = __syncthreads_or(open) == 0;
  }
  if (!settled) return false;
  // kept members in order: thread t counts its contiguous chunk, the chunks are scanned, and every thread
  // writes its kept members at their ranks, up to P
  const int chunk = (n_cand + kNT - 1) / kNT;
  const int i0 = min(tid * chunk, n_cand), i1 = min(i0 + chunk, n_cand);
  int mine = 0;
  for (int i = i0; i < i1; ++i) mine += state[i] == 1;
  int incl = mine;                                     // inclusive scan: lanes by shuffle, then the warps' totals
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s_scan[warp] = incl;
  __syncthreads();
  int before = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kNT / 32; ++w) { const int v = s_scan[w]; if (w < warp) before += v; total += v; }
  int rank = before + incl - mine;
  for (int i = i0; i < i1 && rank < p.n_keep; ++i) {
    if (state[i] == 1) {
      kept_out[rank] = cand[i];
      p.kept_pos[rank] = i;
      if (rank == p.n_keep - 1) *n_examined = i + 1;   // the walk stops here
      ++rank;
    }
  }
  if (tid == 0) *n_kept = min(total, p.n_keep);
  __syncthreads();
  return true;
}

}  // namespace strads
