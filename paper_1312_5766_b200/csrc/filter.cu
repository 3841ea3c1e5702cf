// SAP step 2 / Algorithm 1 "choose a set B1 of <= P coefficients from U such that |x_j^T x_k| < rho":
// greedy first-fit over the candidates in sampling order, on the conflict bits of the Gram kernel.
//
// The walk is a serial chain (whether candidate i is kept depends on every earlier decision).  One CTA
// takes the list 64 positions at a time.  For such a range the candidates not blocked so far are two words
// of the running `blocked` mask, and the conflicts of a member with the other 63 are two words of its
// conflict row (the range is 64-aligned): nothing is searched or compacted.  One warp settles the range in a
// few passes of warp-wide ORs (see below) instead of 64 dependent steps, and the rows of the newly kept
// candidates are then OR-ed into `blocked` for the ranges still to come by the whole CTA.
// The conflict rows are read from shared memory: all of them are brought in once when they fit (a
// candidate window does), otherwise the rows of the range's unblocked members are fetched per range.
#include "strads_internal.cuh"
#include "walk_pairs.cuh"

namespace strads {
namespace {

constexpr int kThreads = 256;
constexpr int kRange = 64;                       // positions decided per step of the walk
constexpr size_t kResidentBytes = 200 * 1024;    // conflict rows of the whole list in shared memory up to this

__host__ __device__ inline int words_of(int n_cand) { return (n_cand + 31) >> 5; }
__host__ __device__ inline int pitch_of(int n_cand) { return words_of(n_cand) | 1; }      // odd: rows start in different banks
__host__ __device__ inline int cand_offset(int n_cand) { return (words_of(n_cand) + 2 + 3) & ~3; }   // after blocked[Wn + 2]
__host__ __device__ inline int rows_offset(int n_cand) { return cand_offset(n_cand) + ((n_cand + 3) & ~3); }   // after s_cand[n_cand]

// n_cand < n_total: the list is only a leading window of the candidates.  If P are kept inside it the result
// is final (the walk never looks further); otherwise window_short is raised and the caller's retry over
// the whole list (launched with only_if_short) replaces the result.
__global__ void __launch_bounds__(kThreads) k_filter(Problem p, const int* __restrict__ cand, int n_cand, int n_total,
                                                      int only_if_short, int resident, int only_if_pending,
                                                      int* __restrict__ kept_out) {
  chain_begin();
  if (only_if_short && !p.st->window_short) return;
  if (only_if_pending && !p.st->walk_pending) return;
  if (n_cand < n_total && p.st->amb_count > (unsigned)p.cap_amb) {
    // dense window whose BF16 screen left more borderline pairs than the list holds: its bits are incomplete;
    // the whole-list retry (which has the 3xTF32 fallback) takes over
    if (threadIdx.x == 0) { p.st->window_short = 1; p.st->route = 1; p.st->amb_count = 0; p.st->edge_count = 0; p.st->edges_off = 0; }
    return;
  }
  if (p.layout == STRADS_CSC && n_cand < n_total && window_skipped(p)) {
    if (threadIdx.x == 0) { p.st->window_short = 1; p.st->route = 1; p.st->edge_count = 0; p.st->edges_off = 0; }   // window attempt skipped: go straight to the whole-list walk
    return;
  }
  extern __shared__ unsigned int sm[];
  const int W = p.mask_words;                    // pitch of the conflict rows in global memory
  const int Wn = words_of(n_cand), Wp = pitch_of(n_cand);
  unsigned int* blocked = sm;                    // [Wn + 2] (two words of slack: a range always reads a pair)
  int* s_cand = reinterpret_cast<int*>(sm + cand_offset(n_cand));   // [n_cand] copy of the list
  unsigned int* rows = sm + rows_offset(n_cand); // resident: [n_cand][Wp]; else the range in flight, [kRange][Wp]
  __shared__ unsigned long long s_keep;          // members of the range in flight that were kept
  __shared__ int s_kept, s_examined, s_done;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) { s_kept = 0; s_examined = n_cand; s_done = 0; }

  if (p.flags & STRADS_FLAG_NO_FILTER) {
    const int nk = min(n_cand, p.n_keep);
    for (int i = tid; i < p.n_keep; i += kThreads) kept_out[i] = i < nk ? cand[i] : -1;
    if (tid == 0) {
      p.st->counts[1] = nk; p.st->counts[2] = nk; p.st->counts[3] = 0; p.st->amb_count = 0; p.st->window_short = 0;
      p.st->route = 0; p.st->walk_pending = 0;
      p.st->edge_count = 0; p.st->edges_off = 0;
    }
    return;
  }

  // ---- The walk from the list of conflicting pairs, when the Gram kernels listed all of them. ----
  bool settled = false;
  const unsigned int n_edges = p.st->edge_count;
  if (!p.st->edges_off && n_edges <= (unsigned)p.cap_edges) {
    __syncthreads();                                                      // s_kept, s_examined are set
    settled = walk_from_pair_list<kThreads>(p, cand, n_cand, n_edges, reinterpret_cast<unsigned char*>(sm), kept_out,
                                            &s_kept, &s_examined);
    __syncthreads();
  }

  for (int w = tid; w < Wn + 2 && !settled; w += kThreads) blocked[w] = 0u;
  const int n_rows = settled ? 0 : n_cand;             // (settled: nothing left for the walk over the bit rows)
  for (int i = tid; i < n_rows; i += kThreads) s_cand[i] = cand[i];
  if (resident && (W & 3) == 0 && Wn <= 64) {
    // all rows at once, 128-bit loads: 8 or 16 lanes per row (one per group of four words), sixteen rows in
    // flight per thread, loads before stores
    const int quads = (Wn + 3) >> 2;                   // (W % 4 == 0: 4 * quads <= W)
    const int lpr_log = quads <= 8 ? 3 : 4, lpr = 1 << lpr_log;
    const int c = tid & (lpr - 1), rstep = kThreads >> lpr_log;
    for (int r0 = tid >> lpr_log; r0 < n_rows; r0 += 16 * rstep) {
      uint4 v[16];
#pragma unroll
      for (int u = 0; u < 16; ++u) {
        const int r = r0 + u * rstep;
        v[u] = make_uint4(0u, 0u, 0u, 0u);
        if (r < n_rows && c < quads) v[u] = __ldcg(reinterpret_cast<const uint4*>(p.conflict + (long long)r * W) + c);
      }
#pragma unroll
      for (int u = 0; u < 16; ++u) {
        const int r = r0 + u * rstep;
        if (r < n_rows && c < quads) {
          unsigned int* dst = rows + r * Wp + 4 * c;
          dst[0] = v[u].x;
          if (4 * c + 1 < Wn) dst[1] = v[u].y;
          if (4 * c + 2 < Wn) dst[2] = v[u].z;
          if (4 * c + 3 < Wn) dst[3] = v[u].w;
        }
      }
    }
  } else if (resident) {
    // all rows at once: independent loads, eight in flight per thread, before any store
    const int total = n_rows * Wn;
    for (int i0 = tid; i0 < total; i0 += 8 * kThreads) {
      unsigned int v[8];
      int at[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = min(i0 + u * kThreads, total - 1);
        const int r = i / Wn, w = i - r * Wn;
        at[u] = r * Wp + w;
        v[u] = __ldcg(p.conflict + (long long)r * W + w);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (i0 + u * kThreads < total) rows[at[u]] = v[u];
    }
  }
  __syncthreads();

  for (int cur = 0; cur < n_rows; cur += kRange) {
    const int m = min(kRange, n_cand - cur);
    const int w0 = cur >> 5;                           // even: the range is words w0, w0 + 1 of every mask
    const unsigned long long valid = m >= 64 ? ~0ull : ((1ull << m) - 1ull);
    const unsigned long long alive0 = ~(((unsigned long long)blocked[w0 + 1] << 32) | blocked[w0]) & valid;
    if (alive0 == 0ull) continue;                      // (uniform) everything here is blocked already
    if (!resident) {
      // rows of the unblocked members, words w0 .. Wn - 1 (earlier words are never looked at again).  One CTA
      // has few loads in flight, so they are 128-bit where the row pitch allows: a task is four consecutive
      // words of one member's row, sixteen tasks in flight per thread, loads before stores.
      if ((W & 3) == 0) {
        // thread -> member tid / 4 and every fourth 128-bit group of its row from tid % 4 on (four lanes read 64
        // consecutive bytes)
        const int q = tid >> 2, v0 = w0 >> 2, vend = (Wn + 3) >> 2;                  // (W % 4 == 0: 4 * vend <= W)
        const bool on = (alive0 >> q) & 1ull;
        const uint4* src = reinterpret_cast<const uint4*>(p.conflict + (long long)(cur + q) * W);
        unsigned int* dst = rows + q * Wp;
        for (int c0 = v0 + (tid & 3); c0 < vend; c0 += 4 * 16) {
          uint4 v[16];
#pragma unroll
          for (int u = 0; u < 16; ++u) {
            const int c = c0 + 4 * u;
            v[u] = make_uint4(0u, 0u, 0u, 0u);
            if (on && c < vend) v[u] = __ldcg(src + c);
          }
#pragma unroll
          for (int u = 0; u < 16; ++u) {
            const int c = c0 + 4 * u;
            if (c < vend) {
              dst[4 * c] = v[u].x;
              if (4 * c + 1 < Wn) dst[4 * c + 1] = v[u].y;
              if (4 * c + 2 < Wn) dst[4 * c + 2] = v[u].z;
              if (4 * c + 3 < Wn) dst[4 * c + 3] = v[u].w;
            }
          }
        }
      } else {
        const int chunks = (Wn - w0 + 31) >> 5, tasks = kRange * chunks;
        for (int t0 = warp; t0 < tasks; t0 += 16 * (kThreads / 32)) {
          unsigned int v[16];
#pragma unroll
          for (int u = 0; u < 16; ++u) {
            const int task = t0 + u * (kThreads / 32);
            const int q = task & (kRange - 1), wd = w0 + ((task >> 6) << 5) + lane;
            v[u] = (task < tasks && wd < Wn && ((alive0 >> q) & 1ull)) ? __ldcg(p.conflict + (long long)(cur + q) * W + wd) : 0u;
          }
#pragma unroll
          for (int u = 0; u < 16; ++u) {
            const int task = t0 + u * (kThreads / 32);
            const int q = task & (kRange - 1), wd = w0 + ((task >> 6) << 5) + lane;
            if (task < tasks && wd < Wn) rows[q * Wp + wd] = v[u];
          }
        }
      }
      __syncthreads();
    }
    // The greedy decision inside the range, by warp 0; lane l holds members l and l + 32 with their conflicts
    // with LATER members (all the Gram kernels guarantee).  Instead of 64 dependent steps it settles the range in
    // passes: members hit by a member kept in the last pass are out; a member that no earlier undecided member
    // conflicts with is kept (all its earlier neighbours are out).  The first undecided member is always kept, so
    // the passes end; with few conflicts two or three do.  Same set as the one-by-one walk.
    if (tid < 32) {
      const unsigned int full = 0xffffffffu;
      const int base = resident ? cur * Wp + w0 : w0;
      const int cva = lane < m ? s_cand[cur + lane] : -1;
      const int cvb = lane + 32 < m ? s_cand[cur + lane + 32] : -1;
      const int ata = base + min(lane, m - 1) * Wp, atb = base + min(lane + 32, m - 1) * Wp;
      const unsigned int later = lane == 31 ? 0u : (full << (lane + 1));
      const unsigned int a_lo = rows[ata] & later, a_hi = rows[ata + 1], b_hi = rows[atb + 1] & later;
      unsigned int und_lo = (unsigned int)alive0, und_hi = (unsigned int)(alive0 >> 32);
      unsigned int keep_lo = 0u, keep_hi = 0u, new_lo = 0u, new_hi = 0u;
      for (int pass = 0; pass < kRange && (und_lo | und_hi) != 0u; ++pass) {
        if (pass > 0) {
          const bool ka = (new_lo >> lane) & 1u, kb = (new_hi >> lane) & 1u;
          und_lo &= ~__reduce_or_sync(full, ka ? a_lo : 0u);
          und_hi &= ~__reduce_or_sync(full, (ka ? a_hi : 0u) | (kb ? b_hi : 0u));
        }
        const bool ua = (und_lo >> lane) & 1u, ub = (und_hi >> lane) & 1u;
        const unsigned int thr_lo = __reduce_or_sync(full, ua ? a_lo : 0u);
        const unsigned int thr_hi = __reduce_or_sync(full, (ua ? a_hi : 0u) | (ub ? b_hi : 0u));
        new_lo = und_lo & ~thr_lo; new_hi = und_hi & ~thr_hi;
        keep_lo |= new_lo; keep_hi |= new_hi;
        und_lo &= ~new_lo; und_hi &= ~new_hi;
      }
      unsigned long long keep = ((unsigned long long)keep_hi << 32) | keep_lo;
      const int nk = s_kept;
      const int room = p.n_keep - nk;
      bool full_now = false;
      if (__popcll(keep) >= room) {                    // stop exactly at P: drop the surplus from the back
        while (__popcll(keep) > room) keep &= ~(1ull << (63 - __clzll(keep)));
        full_now = true;
      }
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int q = lane + 32 * half;
        if ((keep >> q) & 1ull) {
          const int r = __popcll(keep & ((1ull << q) - 1ull));
          kept_out[nk + r] = half ? cvb : cva;
          p.kept_pos[nk + r] = cur + q;
        }
      }
      if (lane == 0) {
        s_keep = keep;
        s_kept = nk + __popcll(keep);
        if (full_now) { s_examined = cur + (63 - __clzll(keep)) + 1; s_done = 1; }
      }
    }
    __syncthreads();
    if (s_done) break;
    // OR the rows of the newly kept candidates into the mask of the ranges still to come.  A lane per mask
    // word (32 consecutive words per trip), warp k takes the members k, k + 8, ... of the range: no reduction
    // across lanes, eight independent reads per trip, and one shared-memory atomic OR per word and warp.
    {
      const unsigned long long keep = s_keep;
      int kr[kRange / 8];
      bool any = false;
#pragma unroll
      for (int u = 0; u < kRange / 8; ++u) {
        const int q = warp + 8 * u;
        const bool k = (keep >> q) & 1ull;
        kr[u] = k ? (resident ? cur + q : q) * Wp : -1;
        any |= k;
      }
      if (any) {
        for (int w = w0 + 2 + lane; w < Wn; w += 32) {
          unsigned int acc = 0u;
#pragma unroll
          for (int u = 0; u < kRange / 8; ++u) acc |= kr[u] >= 0 ? rows[kr[u] + w] : 0u;
          if (acc != 0u) atomicOr(&blocked[w], acc);
        }
      }
    }
    __syncthreads();
  }
  __syncthreads();
  const int nk = s_kept;
  for (int i = nk + tid; i < p.n_keep; i += kThreads) kept_out[i] = -1;
  if (tid == 0) {
    p.st->counts[1] = s_examined; p.st->counts[2] = nk; p.st->counts[3] = 0; p.st->amb_count = 0;
    p.st->edge_count = 0; p.st->edges_off = 0;         // the next Gram starts a new list
    // (the whole-list retry leaves the flag as the window's walk set it: kernels of a parallel branch may still read it)
    if (!only_if_short) p.st->window_short = (nk < p.n_keep && n_cand < n_total) ? 1 : 0;
    if (!only_if_short && !only_if_pending) p.st->route = p.st->window_short;   // (left to it by the window's Gram: stays on the retry branch)
    p.st->walk_pending = 0;
    if (!only_if_short && n_cand < n_total) {          // a window attempt: remember how it went
      if (p.st->window_short) p.st->walk_streak = min(p.st->walk_streak + 1, 16);
      else { p.st->prefer_walk = 0; p.st->walk_streak = 0; }
    }
  }
}

}  // namespace

static size_t filter_smem_bytes(int n_cand, bool* resident) {
  // + 4 words: the pair of words a range reads from the last row may reach one word past it (odd word count)
  const size_t all = ((size_t)rows_offset(n_cand) + (size_t)n_cand * pitch_of(n_cand) + 4) * sizeof(unsigned int);
  *resident = all <= kResidentBytes;
  return *resident ? all : ((size_t)rows_offset(n_cand) + (size_t)kRange * pitch_of(n_cand) + 4) * sizeof(unsigned int);
}

// Kernel-wide attribute: the largest size any handle can need (see prepare_sample).
cudaError_t prepare_filter(const Problem&) {
  bool r;
  size_t most = filter_smem_bytes(STRADS_MAX_CANDIDATES, &r);
  if (most < kResidentBytes) most = kResidentBytes;
  return cudaFuncSetAttribute(k_filter, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most);
}

cudaError_t launch_filter(const Problem& p, const int* cand, int n_cand, int n_total, bool only_if_short, int* kept_out,
                          cudaStream_t s, bool only_if_pending) {
  bool resident;
  size_t smem = filter_smem_bytes(n_cand, &resident);
  const size_t sparse = walk_pairs_smem(n_cand, (unsigned)p.cap_edges);                                          // walk from the pair list
  if (smem < sparse) smem = sparse;
  return launch_chained(k_filter, 1, kThreads, smem, s, p, cand, n_cand, n_total, only_if_short ? 1 : 0, resident ? 1 : 0,
                        only_if_pending ? 1 : 0, kept_out);
}

}  // namespace strads
