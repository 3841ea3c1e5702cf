// SAP step 2, CSC X, when the walk needs the whole candidate list: greedy first-fit that forms conflict
// rows ON DEMAND.  Only the row of a candidate that is kept is ever needed (it tells which later candidates
// it blocks), so with heavy rejection -- skewed rows make most pairs of columns overlap, a few dozen
// candidates are kept out of 16,384 -- forming all P'(P'-1)/2 correlations first would do 100x more merges
// than the walk consults.
//
// One cooperative kernel, one CTA per SM, in batches of 32 candidates.  Every CTA holds the running
// `blocked` mask in shared memory and does the cheap, serial part of a batch itself, identically to all the
// others, so that nothing has to be broadcast:
//   A  pick the next 32 candidates that are not blocked yet;
//   B  stage their columns in shared memory and merge the <= 496 pairs among them;
//   C  decide the batch (who is kept) from those in-batch conflicts;
// then the expensive part is shared out over the grid:
//   D  for every candidate just kept, merge its column against all later unblocked candidates (a warp per
//      32 of them, a lane per pair) and OR the resulting conflict words into the mask in global memory
//      (integer OR: any order gives the same mask);
// one grid-wide barrier, and every CTA reloads the mask.  The barrier is a counter + generation word in
// global memory; every spin has an iteration limit, after which the CTA raises STRADS_STATUS_WAIT_EXPIRED
// and leaves (the launch is cooperative, so all CTAs are resident and the limit is never met in practice).
// The kept list equals that of the full-Gram walk: same correlations (same order of the same products),
// same order of decisions.
#include "strads_internal.cuh"

namespace strads {
namespace {

constexpr int kThreads = 256;
constexpr int kBatch = 32;
constexpr int kColCap = 64;           // entries of a batch member's column staged in shared memory (longer: global)
constexpr int kMaxWords = STRADS_MAX_CANDIDATES / 32;
constexpr unsigned int kSpinLimit = 1u << 26;

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

// (written by other SMs earlier in the same launch: read past L1)
__device__ __forceinline__ WalkColumn load_walk_column(const WalkColumn* at) {
  const longlong2 a = __ldcg(reinterpret_cast<const longlong2*>(at));
  const double2 b = __ldcg(reinterpret_cast<const double2*>(at) + 1);
  WalkColumn col;
  col.q0 = a.x; col.n = (int)(a.y & 0xffffffffll); col.j = (int)(a.y >> 32); col.n2 = b.x; col.unused = 0.0;
  return col;
}

// Grid-wide barrier.  Returns false when the wait gave up (or an earlier one did).
__device__ bool grid_barrier(WalkControl* c, unsigned int n_ctas, unsigned int* status, unsigned int limit) {
  __shared__ int s_ok;
  __syncthreads();
  if (threadIdx.x == 0) {
    bool ok = true;
    __threadfence();
    volatile unsigned int* gen = &c->bar_gen;
    const unsigned int g = *gen;                         // cannot advance before this CTA has arrived
    if (atomicAdd(&c->bar_count, 1u) == n_ctas - 1) {
      c->bar_count = 0;
      __threadfence();
      atomicAdd(&c->bar_gen, 1u);
    } else {
      unsigned int it = 0;
      while (*gen == g && ++it < limit) {}
      if (*gen == g) { ok = false; atomicOr(status, STRADS_STATUS_WAIT_EXPIRED); c->failed = 1; }
    }
    __threadfence();
    if (*reinterpret_cast<volatile int*>(&c->failed)) ok = false;
    s_ok = ok;
  }
  __syncthreads();
  return s_ok != 0;
}

__global__ void __launch_bounds__(kThreads) k_walk_csc(Problem p, const int* __restrict__ cand, int n_cand, int window,
                                                        int only_if_short, int* __restrict__ kept_out) {
  if (only_if_short && !p.st->window_short) return;      // uniform over the grid: nobody reaches a barrier
  // a wait that expired in an earlier launch left the barrier's counter where it was: nothing runs on this handle
  // until strads_recover has cleared it (CTAs that disagree on this bit only meet a barrier that gives up)
  if (p.st->status & STRADS_STATUS_WAIT_EXPIRED) return;
  const unsigned int spin_limit = p.wait_limit ? p.wait_limit : kSpinLimit;
  __shared__ unsigned int blocked[kMaxWords];
  __shared__ int brow[kBatch][kColCap + 1];             // (odd pitch: threads that merge different members' columns
  __shared__ float bval[kBatch][kColCap + 1];           //  read different banks)
  __shared__ int s_pref[kMaxWords + 1];                  // unblocked candidates before each mask word (step D)
  __shared__ int s_wsum[kThreads / 32];
  __shared__ int s_pos[kBatch], s_col[kBatch], s_len[kBatch];
  __shared__ long long s_ptr[kBatch];
  __shared__ double s_n2[kBatch];
  __shared__ unsigned int s_conf[kBatch];
  __shared__ unsigned int s_keep;
  __shared__ int s_m, s_cursor, s_kept, s_examined, s_done;
  WalkControl* c = p.walk_ctl;
  const int W = (n_cand + 31) >> 5;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned int n_ctas = gridDim.x;
  const unsigned int full = 0xffffffffu;
  unsigned int* blocked_g = p.walk_blocked;
  const double rho = (double)p.rho;
  const bool rows_aligned = (reinterpret_cast<unsigned long long>(p.xrow) & 15ull) == 0ull;   // (xv always is)

  for (int w = tid; w < W; w += kThreads) blocked[w] = 0u;
  if (blockIdx.x == 0)
    for (int w = tid; w < W; w += kThreads) blocked_g[w] = 0u;
  // where every candidate's column lies, gathered by the whole grid once (the first barrier publishes it): a merge
  // of step D then finds its column in one access instead of three dependent ones
  for (int a = (int)(blockIdx.x * kThreads) + tid; a < n_cand; a += (int)(n_ctas * kThreads)) {
    WalkColumn col;
    col.j = cand[a];
    col.q0 = p.xptr[col.j];
    col.n = (int)(p.xptr[col.j + 1] - col.q0);
    col.n2 = coupling_n2(p, col.j);
    col.unused = 0.0;
    p.walk_cols[a] = col;
  }
  if (tid == 0) { s_cursor = 0; s_kept = 0; s_examined = n_cand; s_done = 0; }
  bool ok = grid_barrier(c, n_ctas, &p.st->status, spin_limit);       // nobody ORs into the global mask before it is cleared

  while (ok) {
    // ---- A: the next <= 32 candidates at or after the cursor that are not blocked: every thread counts the free
    //      positions of two mask words, a scan over the CTA numbers them, and the first 32 are the batch (late batches
    //      find theirs thousands of positions further on: one warp scanning 1,024 positions per trip took 4 us) ----
    {
      const int cur = s_cursor;
      auto free_from = [&](int w) {                      // unblocked candidates of mask word w at or behind the cursor
        if (w >= W) return 0u;
        unsigned int f = ~blocked[w];
        const int first = w << 5;
        if (first + 32 <= cur) f = 0u;
        else if (first < cur) f &= full << (cur - first);                                   // (a shift of 1 .. 31)
        if (first + 32 > n_cand) f &= first >= n_cand ? 0u : (full >> (first + 32 - n_cand));
        return f;
      };
      unsigned int f0 = free_from(2 * tid), f1 = free_from(2 * tid + 1);
      const int c0 = __popc(f0), c1 = __popc(f1);
      int incl = c0 + c1;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(full, incl, o);
        if (lane >= o) incl += v;
      }
      if (lane == 31) s_wsum[warp] = incl;
      __syncthreads();
      int before = 0, total = 0;
#pragma unroll
      for (int k = 0; k < kThreads / 32; ++k) { const int v = s_wsum[k]; if (k < warp) before += v; total += v; }
      int idx = before + incl - c0 - c1;
      for (; f0 != 0u && idx < kBatch; f0 &= f0 - 1u, ++idx) s_pos[idx] = ((2 * tid) << 5) + __ffs((int)f0) - 1;
      idx = before + incl - c1;
      for (; f1 != 0u && idx < kBatch; f1 &= f1 - 1u, ++idx) s_pos[idx] = ((2 * tid + 1) << 5) + __ffs((int)f1) - 1;
      if (tid == 0) s_m = min(kBatch, total);
      if (tid < 32) s_conf[tid] = 0u;
    }
    __syncthreads();
    const int m = s_m;
    if (m == 0) break;                                 // list exhausted (the same in every CTA)

    // ---- B: stage the members' columns, all at once (a thread per member finds the column, then eight threads per
    //      member copy it: three memory round trips for the whole batch), then the pairs among them ----
    if (tid < m) {
      const WalkColumn col = load_walk_column(p.walk_cols + s_pos[tid]);
      s_col[tid] = col.j; s_ptr[tid] = col.q0; s_len[tid] = col.n; s_n2[tid] = col.n2;
    }
    __syncthreads();
    {
      const int q = tid >> 3;
      if (q < m && s_len[q] <= kColCap) {
        const long long a0 = s_ptr[q];
        for (int e = tid & 7; e < s_len[q]; e += 8) { brow[q][e] = __ldg(p.xrow + a0 + e); bval[q][e] = __ldg(p.xv + a0 + e); }
      }
    }
    __syncthreads();
    {
      // the m (m - 1) / 2 pairs (qa < qb) in turn over the threads: two per thread for a full batch, side by side,
      // one step of each per trip (the steps of one merge depend on each other, those of different merges do not)
      constexpr int kSide = 2;
      const int n_pairs = m * (m - 1) / 2;
      for (int p0 = tid; p0 < n_pairs; p0 += kSide * kThreads) {
        int qas[kSide], qbs[kSide], nas[kSide], nbs[kSide], ii[kSide], kk[kSide];
        float dots[kSide];
        bool staged = true;
#pragma unroll
        for (int u = 0; u < kSide; ++u) {
          int left = p0 + u * kThreads;
          const bool on = left < n_pairs;
          int qa = 0;
          if (on) while (left >= m - 1 - qa) { left -= m - 1 - qa; ++qa; }     // pair number -> (qa, qb), rows of m-1, m-2, ...
          qas[u] = qa; qbs[u] = on ? qa + 1 + left : qa;
          nas[u] = on ? s_len[qa] : 0; nbs[u] = on ? s_len[qbs[u]] : 0;
          staged = staged && nas[u] <= kColCap && nbs[u] <= kColCap;
          ii[u] = 0; kk[u] = 0; dots[u] = 0.f;
        }
        if (staged) {
          bool any = true;
          while (any) {
            any = false;
#pragma unroll
            for (int u = 0; u < kSide; ++u) {
              const bool on = ii[u] < nas[u] && kk[u] < nbs[u];
              const int i = on ? ii[u] : 0, k = on ? kk[u] : 0;
              const int ra = brow[qas[u]][i], rb = brow[qbs[u]][k];
              if (on && ra == rb) dots[u] = fmaf(bval[qas[u]][i], bval[qbs[u]][k], dots[u]);   // (the values only then)
              ii[u] += (on && ra <= rb) ? 1 : 0;
              kk[u] += (on && rb <= ra) ? 1 : 0;
              any = any || on;
            }
          }
        } else {                                       // a column too long for its slot: plain merges from global memory
#pragma unroll
          for (int u = 0; u < kSide; ++u) {
            const int qa = qas[u], qb = qbs[u], na = nas[u], nb = nbs[u];
            const int* ar = na <= kColCap ? brow[qa] : p.xrow + s_ptr[qa];
            const float* av = na <= kColCap ? bval[qa] : p.xv + s_ptr[qa];
            const int* br = nb <= kColCap ? brow[qb] : p.xrow + s_ptr[qb];
            const float* bv = nb <= kColCap ? bval[qb] : p.xv + s_ptr[qb];
            dots[u] = sparse_dot_arrays(ar, av, na, br, bv, nb);
          }
        }
#pragma unroll
        for (int u = 0; u < kSide; ++u) {
          const double den = sqrt(s_n2[qas[u]] * s_n2[qbs[u]]);
          if (nbs[u] > 0 && nas[u] > 0 && den > 0.0 && fabs((double)dots[u]) >= rho * den) atomicOr(&s_conf[qas[u]], 1u << qbs[u]);
        }
      }
    }
    __syncthreads();

    // ---- C: decide the batch (warp 0, lane = member; the same in every CTA).  Passes of warp-wide ORs: members hit
    //      by one kept in the last pass are out; a member no earlier undecided member conflicts with is kept. ----
    if (tid < 32) {
      const unsigned int valid = m >= 32 ? full : ((1u << m) - 1u);
      const unsigned int mine = s_conf[lane];          // conflicts with LATER members only
      unsigned int und = valid, keep = 0u, fresh = 0u;
      for (int pass = 0; pass < kBatch && und != 0u; ++pass) {
        if (pass > 0) und &= ~__reduce_or_sync(full, ((fresh >> lane) & 1u) ? mine : 0u);
        const unsigned int thr = __reduce_or_sync(full, ((und >> lane) & 1u) ? mine : 0u);
        fresh = und & ~thr;
        keep |= fresh;
        und &= ~fresh;
      }
      const int nk = s_kept;
      const int room = p.n_keep - nk;
      bool done = false;
      if (__popc(keep) >= room) {                      // stop exactly at P: drop the surplus from the back
        while (__popc(keep) > room) keep &= ~(1u << (31 - __clz(keep)));
        done = true;
      }
      if (blockIdx.x == 0 && ((keep >> lane) & 1u)) kept_out[nk + __popc(keep & ((1u << lane) - 1u))] = s_col[lane];
      if (lane == 0) {
        s_keep = keep;
        s_kept = nk + __popc(keep);
        if (done) { s_examined = s_pos[31 - __clz(keep)] + 1; s_done = 1; }
        else s_cursor = s_pos[m - 1] + 1;
      }
    }
    __syncthreads();
    if (s_done) break;                                 // P kept: what they block no longer matters

    // ---- D: the kept members' conflicts with the later candidates that are not blocked yet, shared out over the
    //      grid with a lane per (candidate, kept member) pair.  Every CTA numbers the unblocked candidates behind the
    //      first kept member from its own copy of the mask (the same in all CTAs), so that pair number L of the grid is
    //      member L / U against the (L mod U)-th of them: late batches, in which a dozen members meet a few hundred
    //      survivors, still use every lane.  A lane fetches its candidate's rows and values together and merges them
    //      against the member's column in shared memory. ----
    {
      const unsigned int keep = s_keep;
      const int n_new = __popc(keep);
      const int first_pos = s_pos[__ffs(keep) - 1];      // candidates at or before the first kept member are not touched
      auto free_word = [&](int w) {                      // unblocked candidates of mask word w behind first_pos
        unsigned int f = ~blocked[w];
        const int first = w << 5;
        if (first + 31 <= first_pos) f = 0u;
        else if (first <= first_pos) f &= full << (first_pos - first + 1);     // (a shift of 1 .. 31)
        if (first + 32 > n_cand) f &= first >= n_cand ? 0u : (full >> (first + 32 - n_cand));
        return f;
      };
      // exclusive prefix of the per-word counts: two words per thread (W <= 512), warp scan, then the warps' totals
      int c0 = 0, c1 = 0;
      if (2 * tid < W) c0 = __popc(free_word(2 * tid));
      if (2 * tid + 1 < W) c1 = __popc(free_word(2 * tid + 1));
      int incl = c0 + c1;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(full, incl, o);
        if (lane >= o) incl += v;
      }
      if (lane == 31) s_wsum[warp] = incl;
      __syncthreads();
      int before = 0, U = 0;
#pragma unroll
      for (int k = 0; k < kThreads / 32; ++k) { const int v = s_wsum[k]; if (k < warp) before += v; U += v; }
      const int excl = before + incl - c0 - c1;
      if (2 * tid < W) s_pref[2 * tid] = excl;
      if (2 * tid + 1 < W) s_pref[2 * tid + 1] = excl + c0;
      if (tid == 0) s_pref[W] = U;
      __syncthreads();
      const long long pairs = (long long)U * n_new;
      const long long n_lanes = (long long)n_ctas * kThreads;
      // (warp g of the grid = warp g / n_ctas of CTA g mod n_ctas: a few hundred pairs spread over all SMs instead of
      //  filling the first few CTAs)
      for (long long L = ((long long)warp * n_ctas + blockIdx.x) * 32 + lane; L < pairs; L += n_lanes) {
        const int k = (int)(L / U), u = (int)(L - (long long)k * U);
        int lo = 0, hi = W;                              // the word that holds the u-th unblocked candidate
        while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (s_pref[mid] <= u) lo = mid; else hi = mid; }
        const int b = (lo << 5) + nth_set_bit(free_word(lo), u - s_pref[lo]);
        const int q = nth_set_bit(keep, k);
        if (s_pos[q] >= b) continue;                     // the member comes later in the list: it cannot block b
        const WalkColumn cb = load_walk_column(p.walk_cols + b);
        const long long q0 = cb.q0;
        const int nb = cb.n;
        const double den = sqrt(s_n2[q] * cb.n2);
        const int na = s_len[q];
        const int* ar = na <= kColCap ? brow[q] : p.xrow + s_ptr[q];
        const float* av = na <= kColCap ? bval[q] : p.xv + s_ptr[q];
        float dot;
        const int need = (int)(q0 & 3) + nb;               // entries of the aligned groups of four that hold column b
        if (!rows_aligned) dot = nb <= 24 ? sparse_dot_fetched<24>(ar, av, na, p, q0, nb) : sparse_dot_fetched<32>(ar, av, na, p, q0, nb);
        else if (need <= 20) dot = sparse_dot_fetched4<5>(ar, av, na, p, q0, nb);
        else if (need <= 28) dot = sparse_dot_fetched4<7>(ar, av, na, p, q0, nb);
        else if (need <= 36) dot = sparse_dot_fetched4<9>(ar, av, na, p, q0, nb);
        else dot = sparse_dot_arrays(ar, av, na, p.xrow + q0, p.xv + q0, nb);
        if (den > 0.0 && fabs((double)dot) >= rho * den) atomicOr(&blocked_g[b >> 5], 1u << (b & 31));
      }
    }
    ok = grid_barrier(c, n_ctas, &p.st->status, spin_limit);
    if (!ok) break;
    for (int w = tid; w < W; w += kThreads) blocked[w] = __ldcg(&blocked_g[w]);
    __syncthreads();
  }

  if (blockIdx.x == 0) {
    __syncthreads();
    const int nk = s_kept;
    for (int i = nk + tid; i < p.n_keep; i += kThreads) kept_out[i] = -1;
    if (tid == 0) {
      p.st->counts[1] = s_examined; p.st->counts[2] = nk; p.st->counts[3] = 0;
      p.st->amb_count = 0; p.st->window_short = 0; p.st->prefer_walk = 1;
      // would a window of the first `window` candidates have done?  (window_skipped consults this in the next round)
      p.st->window_hopeless = (nk == p.n_keep && s_examined <= window) ? 0 : 1;
      c->failed = 0;
    }
  }
}

}  // namespace

// The cooperative grid for this device: one CTA per SM.
cudaError_t prepare_walk_csc(const Problem& p, int* grid_out) {
  int per_sm = 0;
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_walk_csc, kThreads, 0);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  // one CTA per SM: the serial part of a batch is the same in every CTA, and the grid-wide part is short, so the
  // second CTA of an SM only slowed its neighbour and the barrier down (c5 walk 131 -> 117 us)
  *grid_out = p.sm_count * (per_sm < 1 ? per_sm : 1);
  return cudaSuccess;
}

cudaError_t launch_walk_csc(const Problem& p, const int* cand, int n_cand, int window, int grid, bool only_if_short, int* kept_out,
                            cudaStream_t s) {
  Problem q = p;
  int ois = only_if_short ? 1 : 0;
  void* args[] = {&q, &cand, &n_cand, &window, &ois, &kept_out};
  return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(k_walk_csc), dim3(grid), dim3(kThreads), args, 0, s);
}

}  // namespace strads
