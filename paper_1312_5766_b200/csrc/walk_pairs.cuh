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
//
// The CTA that runs this has the rest of the grid idle behind it, and with so few warps every instruction waits
// for the one before it (time stamps: ~1 us per pass and per scan when each was a loop over all candidates with
// its own barriers), so the work is cut to short chains: only the second members of listed pairs are ever
// undecided, the passes touch nothing but the pairs, and the kept sequence is numbered from warp ballots.
#pragma once
#include "strads_internal.cuh"

namespace strads {

constexpr int kSparsePasses = 24;

// Bytes of shared memory the walk needs for n_cand candidates and n_edges listed pairs.
__host__ __device__ inline size_t walk_pairs_smem(int n_cand, unsigned int n_edges) {
  const size_t bytes = ((size_t)n_cand + 15) & ~(size_t)15, words = ((size_t)n_cand + 31) / 32 + 1;
  return 3 * bytes + 2 * sizeof(unsigned int) * words + sizeof(unsigned int) * (size_t)n_edges;
}

// Returns whether the walk was settled (uniform over the CTA).  If so, kept_out[0 .. *n_kept) and
// p.kept_pos[0 .. *n_kept) hold the kept coefficients and their positions in the list, and *n_examined the
// position after the P-th kept one (left alone when fewer than P are kept).  n_kept / n_examined: shared memory.
template <int kNT>
__device__ bool walk_from_pair_list(const Problem& p, const int* __restrict__ cand, int n_cand, unsigned int n_edges,
                                    unsigned char* sm, int* __restrict__ kept_out, int* n_kept, int* n_examined) {
  const int tid = threadIdx.x, lane = tid & 31;
  const size_t bytes = ((size_t)n_cand + 15) & ~(size_t)15;
  const int n_words = (n_cand + 31) / 32;
  unsigned char* state = sm;                                              // 0 undecided, 1 kept, 2 out
  unsigned char* hit = state + bytes;                                     // has a kept earlier neighbour
  unsigned char* pend = hit + bytes;                                      // pass + 1 of the last pass that saw an undecided earlier neighbour
  unsigned int* wbits = reinterpret_cast<unsigned int*>(pend + bytes);    // [n_words] kept flags of 32 consecutive candidates
  unsigned int* wpre = wbits + n_words + 1;                               // [n_words + 1] kept members before each word
  unsigned int* e = wpre + n_words + 1;
  // the candidates this thread will write out if they are kept (positions tid, tid + kNT, ...), asked for now
  constexpr int kAhead = 4;
  int cv[kAhead];
#pragma unroll
  for (int u = 0; u < kAhead; ++u) cv[u] = tid + u * kNT < n_cand ? cand[tid + u * kNT] : 0;
  for (int i = tid; i < n_cand; i += kNT) state[i] = 1;                    // kept unless a listed pair says otherwise
  for (unsigned int k = tid; k < n_edges; k += kNT) e[k] = __ldcg(p.edges + k);
  __syncthreads();
  if (n_edges > 0) {
    for (unsigned int k = tid; k < n_edges; k += kNT) {                   // (several threads may store the same values: benign)
      const int b = (int)(e[k] & 0xffffu);
      state[b] = 0; hit[b] = 0; pend[b] = 0;
    }
    __syncthreads();
    bool settled = false;
    for (int pass = 0; pass < kSparsePasses && !settled; ++pass) {
      const unsigned char mark = (unsigned char)(pass + 1);
      for (unsigned int k = tid; k < n_edges; k += kNT) {
        const int a = (int)(e[k] >> 16), b = (int)(e[k] & 0xffffu);
        if (state[b] == 0) {
          const unsigned char sa = state[a];
          if (sa == 1) hit[b] = 1;
          else if (sa == 0) pend[b] = mark;
        }
      }
      __syncthreads();
      int open = 0;
      for (unsigned int k = tid; k < n_edges; k += kNT) {                 // every thread that shares b reads the same and stores the same
        const int b = (int)(e[k] & 0xffffu);
        if (state[b] == 0) {
          if (hit[b]) state[b] = 2;
          else if (pend[b] != mark) state[b] = 1;
          else open = 1;
        }
      }
      settled = __syncthreads_or(open) == 0;
    }
    if (!settled) return false;
  }
  // kept members in order: a ballot per 32 consecutive candidates, one warp numbers the words, and every thread
  // writes the kept candidates it looked at, at their ranks, up to P
  for (int i0 = tid - lane; i0 < n_cand; i0 += kNT) {
    const int i = i0 + lane;
    const unsigned int word = __ballot_sync(0xffffffffu, i < n_cand && state[i] == 1);
    if (lane == 0) wbits[i0 >> 5] = word;
  }
  __syncthreads();
  if (tid < 32) {
    unsigned int carry = 0u;
    for (int w0 = 0; w0 < n_words; w0 += 32) {
      const int w = w0 + lane;
      const unsigned int c = w < n_words ? (unsigned int)__popc(wbits[w]) : 0u;
      unsigned int incl = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      if (w < n_words) wpre[w] = carry + incl - c;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) wpre[n_words] = carry;
  }
  __syncthreads();
  int u = 0;
  for (int i = tid; i < n_cand; i += kNT, ++u) {
    const unsigned int word = wbits[i >> 5];
    if ((word >> lane) & 1u) {                             // (i and tid have the same lane: kNT is a multiple of 32)
      const int rank = (int)wpre[i >> 5] + __popc(word & ((1u << lane) - 1u));
      if (rank < p.n_keep) {
        int c;
        switch (u) { case 0: c = cv[0]; break; case 1: c = cv[1]; break; case 2: c = cv[2]; break; case 3: c = cv[3]; break; default: c = cand[i]; }
        kept_out[rank] = c;
        p.kept_pos[rank] = i;
        if (rank == p.n_keep - 1) *n_examined = i + 1;     // the walk stops here
      }
    }
  }
  if (tid == 0) *n_kept = min((int)wpre[n_words], p.n_keep);
  __syncthreads();
  return true;
}

}  // namespace strads
