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

// Position of the n-th (0-based) set bit of x; popc(x) > n.
__device__ __forceinline__ int nth_set_bit(unsigned int x, int n) {
  int at = 0;
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) {
    const int c = __popc(x & ((1u << s) - 1u));
    if (n >= c) { n -= c; x >>= s; at += s; }
  }
  return at;
}

// n_cand < n_total: the list is only a leading window of the candidates.  If P are kept inside it the result
// is final (the walk never looks further); otherwise window_short is raised and the caller's retry over
// the whole list (launched with only_if_short) replaces the result.
__global__ void __launch_bounds__(kThreads) k_filter(Problem p, const int* __restrict__ cand, int n_cand, int n_total,
                                                      int only_if_short, int* __restrict__ kept_out) {
  chain_begin();
  if (only_if_short && !p.st->window_short) return;
  if (n_cand < n_total && p.st->amb_count > (unsigned)p.cap_amb) {
    // dense window whose TF32 screen left more borderline pairs than the list holds: its bits are incomplete;
    // the whole-list retry (which has the 3xTF32 fallback) takes over
    if (threadIdx.x == 0) { p.st->window_short = 1; p.st->amb_count = 0; }
    return;
  }
  if (p.layout == STRADS_CSC && n_cand < n_total && p.st->prefer_walk && ((p.st->round / (unsigned)p.part_count) & 63ull) != 0) {
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
  __shared__ unsigned long long s_conf[kBatch];  // per batch member: conflicts with later members
  __shared__ int s_krow[kBatch], s_kfirst[kBatch], s_nnew;   // newly kept: row offset in `rows`, first valid word
  const int tid = threadIdx.x, lane = tid & 31;
  int G = 1;                                     // threads per mask word in step 4 (a power of two, G * W <= kThreads)
  while (G < 32 && 2 * G * W <= kThreads) G <<= 1;

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
        // slot s of the batch takes the (s - m)-th free position of these 32 words: lane s (and s + 32) finds
        // the word that holds it from the prefix counts, then the bit inside the word
        const int excl = incl - cnt;
#pragma unroll
        for (int half = 0; half < kBatch / 32; ++half) {
          const int slot = lane + 32 * half;
          const int want = slot - m;                   // rank among the free positions found in this sweep
          int wi = 0;                                  // first lane whose inclusive count exceeds `want`
#pragma unroll
          for (int step = 16; step > 0; step >>= 1)
            if (__shfl_sync(0xffffffffu, incl, wi + step - 1) <= want) wi += step;
          wi = min(wi, 31);
          const int ex = __shfl_sync(0xffffffffu, excl, wi);
          const unsigned int word = __shfl_sync(0xffffffffu, freew, wi);
          if (want >= 0 && want < total && slot < kBatch)
            pos[slot] = (((cur >> 5) + wi) << 5) + nth_set_bit(word, want - ex);
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
    // 3a. the conflicts of batch member q with the LATER members, as a 64-bit word: four threads per member,
    //     16 of the 64 bits each (a row is valid from its own word on; fixed trip count so that the reads overlap)
    {
      static_assert(kThreads == 4 * kBatch, "four threads per batch member");
      const int q = tid >> 2, part = tid & 3;
      const int my_row = min(q, m - 1) * Ws;
      unsigned int bits = 0u;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int pb = pos[min(part * 16 + i, m - 1)];
        bits |= ((rows[my_row + (pb >> 5)] >> (pb & 31)) & 1u) << i;
      }
      unsigned long long mine = (unsigned long long)bits << (16 * part);
      mine |= __shfl_xor_sync(0xffffffffu, mine, 1);
      mine |= __shfl_xor_sync(0xffffffffu, mine, 2);
      const unsigned long long valid = m >= 64 ? ~0ull : ((1ull << m) - 1ull);
      const unsigned long long later = q >= 63 ? 0ull : ~((2ull << q) - 1ull);
      if (part == 0) s_conf[q] = q < m ? (mine & valid & later) : 0ull;
    }
    __syncthreads();
    // 3b. the greedy decision inside the batch: 64 steps of register arithmetic (warp 0; every lane computes the same)
    if (tid < 32) {
      const unsigned long long valid = m >= 64 ? ~0ull : ((1ull << m) - 1ull);
      unsigned long long alive = valid, keep = 0ull;
      unsigned long long cq[kBatch];                   // all 64 words into registers first: the loads do not depend
#pragma unroll                                         // on the chain below and overlap
      for (int q = 0; q < kBatch; ++q) cq[q] = s_conf[q];
#pragma unroll
      for (int q = 0; q < kBatch; ++q)
        if ((alive >> q) & 1ull) { keep |= 1ull << q; alive &= ~cq[q]; }
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
#pragma unroll
      for (int half = 0; half < 2; ++half) {           // compact list of the newly kept rows for step 4
        const int q = lane + 32 * half;
        if ((keep >> q) & 1ull) {
          const int r = __popcll(keep & ((1ull << q) - 1ull));
          s_krow[r] = q * Ws;
          s_kfirst[r] = pos[q] >> 5;
        }
      }
      if (lane == 0) {
        s_nnew = __popcll(keep);
        s_kept = nk + __popcll(keep);
        if (full) { s_examined = pos[63 - __clzll(keep)] + 1; s_done = 1; }
        else s_cursor = pos[m - 1] + 1;
      }
    }
    __syncthreads();
    if (s_done) break;
    // 4. OR the rows of the newly kept candidates into the mask (a row is valid from its own word on).
    //    G threads per mask word share the rows between them (all loads unconditional and independent),
    //    then combine with shuffles.
    const int n_new = s_nnew;
    for (int base = 0; base < W; base += kThreads / G) {
      const int w = base + tid / G, sub = tid % G;
      unsigned int acc = 0u;
      if (w < W) {
        for (int r0 = sub; r0 < n_new; r0 += 8 * G) {
          int kf[8];
          unsigned int v[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int r = min(r0 + i * G, n_new - 1);  // past the end: the last row again (harmless)
            kf[i] = s_kfirst[r];
            v[i] = rows[s_krow[r] + w];
          }
#pragma unroll
          for (int i = 0; i < 8; ++i) acc |= w >= kf[i] ? v[i] : 0u;
        }
      }
      for (int o = G >> 1; o > 0; o >>= 1) acc |= __shfl_xor_sync(0xffffffffu, acc, o);
      if (w < W && sub == 0) blocked[w] |= acc;
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
  return launch_chained(k_filter, 1, kThreads, filter_smem_bytes(p), s, p, cand, n_cand, n_total, only_if_short ? 1 : 0, kept_out);
}

}  // namespace strads
