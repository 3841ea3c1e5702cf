// SAP step 2 / Algorithm 1 "choose a set B1 of <= P coefficients from U such that |x_j^T x_k| < rho":
// greedy first-fit over the candidates in sampling order, on the conflict bits of the Gram kernel.
//
// The walk is a serial chain (whether candidate i is kept depends on every earlier decision), and each
// keep needs the conflict row of the kept candidate: a dependent memory access.  To take that latency
// off the chain, one CTA works in batches of 64: the next 64 still-unblocked candidates (the only ones
// that can be kept next) are found with a warp scan, their conflict rows are fetched together into
// shared memory, a thread per candidate extracts its conflicts with the other 63 into one 64-bit word,
// and the greedy decision inside the batch is then 64 steps of register arithmetic.  The rows of the
// newly kept candidates are OR-ed into the running `blocked` mask by the whole CTA.
#include "strads_internal.cuh"

namespace strads {
namespace {

constexpr int kThreads = 256;
constexpr int kBatch = 64;          // candidates decided per batch (two per lane of the deciding warp)

// n_cand < n_total: the list is only a leading window of the candidates.  If P are kept inside it the result
// is final (the walk never looks further); otherwise window_short is raised and the caller's retry over
// the whole list (launched with only_if_short) replaces the result.
__global__ void __launch_bounds__(kThreads) k_filter(Problem p, const int* __restrict__ cand, int n_cand, int n_total,
                                                      int only_if_short, int* __restrict__ kept_out) {
  if (only_if_short && !p.st->window_short) return;
  if (n_cand < n_total && p.st->amb_count > (unsigned)p.cap_amb) {
    // dense window whose TF32 screen left more borderline pairs than the list holds: its bits are incomplete;
    // the whole-list retry (which has the 3xTF32 fallback) takes over
    if (threadIdx.x == 0) { p.st->window_short = 1; p.st->amb_count = 0; }
    return;
  }
  if (p.layout == STRADS_CSC && n_cand < n_total && p.st->prefer_walk && (p.st->round & 63ull) != 0) {
    if (threadIdx.x == 0) p.st->window_short = 1;    // window attempt skipped: go straight to the whole-list walk
    return;
  }
  extern __shared__ unsigned int sm[];
  const int W = p.mask_words;
  const int Ws = W | 1;                          // odd row pitch: column reads of `rows` hit 32 different banks
  unsigned int* blocked = sm;                    // [W]
  unsigned int* rows = sm + W;                   // [kBatch][Ws]
  __shared__ int pos[kBatch];                    // positions (in the candidate list) of the batch
  __shared__ int cval[kBatch];                   // cand[pos[.]]
  __shared__ int s_m, s_cursor, s_kept, s_examined, s_done;
  __shared__ unsigned long long s_keepmask;
  __shared__ unsigned long long s_conf[kBatch];  // per batch member: conflicts with later members
  const int tid = threadIdx.x, lane = tid & 31;

  for (int w = tid; w < W; w += kThreads) blocked[w] = 0u;
  if (tid == 0) { s_cursor = 0; s_kept = 0; s_examined = 0; s_done = 0; }
  __syncthreads();

  if (p.flags & STRADS_FLAG_NO_FILTER) {
    const int nk = min(n_cand, p.n_keep);
    for (int i = tid; i < p.n_keep; i += kThreads) kept_out[i] = i < nk ? cand[i] : -1;
    if (tid == 0) { p.st->counts[1] = nk; p.st->counts[2] = nk; p.st->counts[3] = 0; p.st->amb_count = 0; p.st->window_short = 0; }
    return;
  }

  while (true) {
    // 1. the next <= kBatch candidates at or after the cursor that are not blocked yet (warp 0)
    if (tid < 32) {
      int m = 0;
      int cur = s_cursor;
      while (cur < n_cand && m < kBatch) {
        const int wbase = (cur >> 5) + lane;           // 32 mask words at a time, one per lane
        unsigned int freew = 0u;
        if (wbase < W) {
          freew = ~blocked[wbase];
          const int first = wbase << 5;
          if (first < cur) freew &= 0xffffffffu << (cur - first);                         // only lane 0 can be cut
          if (first + 32 > n_cand) freew &= first >= n_cand ? 0u : (0xffffffffu >> (first + 32 - n_cand));
        }
        const int cnt = __popc(freew);
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += v;
        }
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        int slot = m + incl - cnt;                     // where this lane's first free position goes
        unsigned int fw = freew;
        while (fw && slot < kBatch) {
          const int b = __ffs(fw) - 1;
          fw &= fw - 1;
          pos[slot++] = (wbase << 5) + b;
        }
        m = min(kBatch, m + total);
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
    // 2. fetch their conflict rows (and their coefficient indices) together.  Loads first, stores after:
    //    a store to `rows` between two loads would order them and cost one memory round trip per word.
    if (tid < m) cval[tid] = cand[pos[tid]];         // (kBatch <= kThreads)
    {
      const int warp = tid >> 5;                       // warp w fetches rows w, w + 8, ..., w + 56
      const unsigned int* src[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) src[u] = p.conflict + (long long)pos[min(warp + 8 * u, m - 1)] * W;
      for (int w0 = lane; w0 < W; w0 += 32) {
        unsigned int v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = __ldcg(src[u] + w0);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int r = warp + 8 * u;
          if (r < m) rows[r * Ws + w0] = v[u];
        }
      }
    }
    __syncthreads();
    // 3a. thread q < 64: the conflicts of batch member q with the LATER members, as a 64-bit word
    //     (a row is valid from its own word on; fixed trip count so that the reads overlap)
    if (tid < kBatch) {
      const int my_row = min(tid, m - 1) * Ws;
      unsigned long long mine = 0ull;
#pragma unroll 16
      for (int b = 0; b < kBatch; ++b) {
        const int pb = pos[min(b, m - 1)];
        mine |= (unsigned long long)((rows[my_row + (pb >> 5)] >> (pb & 31)) & 1u) << b;
      }
      const unsigned long long valid = m >= 64 ? ~0ull : ((1ull << m) - 1ull);
      const unsigned long long later = tid >= 63 ? 0ull : ~((2ull << tid) - 1ull);
      s_conf[tid] = tid < m ? (mine & valid & later) : 0ull;
    }
    __syncthreads();
    // 3b. the greedy decision inside the batch: 64 steps of register arithmetic (warp 0; every lane computes the same)
    if (tid < 32) {
      const unsigned long long valid = m >= 64 ? ~0ull : ((1ull << m) - 1ull);
      unsigned long long alive = valid, keep = 0ull;
#pragma unroll 16
      for (int q = 0; q < kBatch; ++q) {
        const unsigned long long cq = s_conf[q];
        if ((alive >> q) & 1ull) { keep |= 1ull << q; alive &= ~cq; }
      }
      const int nk = s_kept;
      const int room = p.n_keep - nk;
      bool full = false;
      if (__popcll(keep) >= room) {                    // stop exactly at P: drop the surplus from the back
        while (__popcll(keep) > room) keep &= ~(1ull << (63 - __clzll(keep)));
        full = true;
      }
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int q = lane + 32 * half;
        if ((keep >> q) & 1ull) {
          const int slot = nk + __popcll(keep & ((1ull << q) - 1ull));
          kept_out[slot] = cval[q];
          p.kept_pos[slot] = pos[q];
        }
      }
      if (lane == 0) {
        s_keepmask = keep;
        s_kept = nk + __popcll(keep);
        if (full) { s_examined = pos[63 - __clzll(keep)] + 1; s_done = 1; }
        else s_cursor = pos[m - 1] + 1;
      }
    }
    __syncthreads();
    if (s_done) break;
    // 4. OR the rows of the newly kept candidates into the mask (a row is valid from its own word on)
    //    Four threads share a word, each takes 16 of the 64 batch members; reads are unconditional so that they overlap.
    const unsigned long long keep = s_keepmask;
    for (int u = tid; u < 4 * W; u += kThreads) {
      const int w = u >> 2, q0 = (u & 3) * 16;
      unsigned int acc = 0u;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int q = q0 + i;
        const unsigned int v = rows[min(q, m - 1) * Ws + w];
        const bool use = ((keep >> q) & 1ull) && w >= (pos[min(q, m - 1)] >> 5);
        acc |= use ? v : 0u;
      }
      if (acc) atomicOr(&blocked[w], acc);
    }
    __syncthreads();
  }
  __syncthreads();
  const int nk = s_kept;
  for (int i = nk + tid; i < p.n_keep; i += kThreads) kept_out[i] = -1;
  if (tid == 0) {
    p.st->counts[1] = s_examined; p.st->counts[2] = nk; p.st->counts[3] = 0; p.st->amb_count = 0;
    p.st->window_short = (!only_if_short && nk < p.n_keep && n_cand < n_total) ? 1 : 0;
    if (!only_if_short && n_cand < n_total && !p.st->window_short) p.st->prefer_walk = 0;
  }
}

}  // namespace

size_t filter_smem_bytes(const Problem& p) {
  return ((size_t)p.mask_words + (size_t)kBatch * (p.mask_words | 1)) * sizeof(unsigned int);
}

// Kernel-wide attribute: the largest size any handle can need (see prepare_sample).
cudaError_t prepare_filter(const Problem&) {
  constexpr int kMaxWords = STRADS_MAX_CANDIDATES / 32;
  return cudaFuncSetAttribute(k_filter, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)((kMaxWords + kBatch * (kMaxWords | 1)) * sizeof(unsigned int)));
}

cudaError_t launch_filter(const Problem& p, const int* cand, int n_cand, int n_total, bool only_if_short, int* kept_out,
                          cudaStream_t s) {
  k_filter<<<1, kThreads, filter_smem_bytes(p), s>>>(p, cand, n_cand, n_total, only_if_short ? 1 : 0, kept_out);
  return cudaGetLastError();
}

}  // namespace strads
