// SAP step 2, CSC X, when the walk needs the whole candidate list: greedy first-fit that forms conflict
// rows ON DEMAND.  Only the row of a candidate that is about to be kept is ever needed (it tells which
// later candidates it blocks), so with heavy rejection -- skewed rows make most pairs of columns overlap,
// a few dozen candidates are kept out of 16,384 -- forming all P'(P'-1)/2 correlations first would do
// 100x more merges than the walk consults.
//
// One cooperative kernel, a few CTAs per SM, in batches of 32 like k_filter:
//   A  CTA 0 picks the next 32 candidates that are not blocked yet;
//   B  all CTAs compute those 32 conflict rows (a row: the candidate's column, staged in shared memory,
//      merged against every later candidate's column; one lane per pair, one ballot per mask word);
//   C  CTA 0 decides the batch in order with register arithmetic and ORs the rows of the newly kept
//      candidates into the running mask;
// with a grid-wide barrier between the phases.  The barrier is a counter + generation word in global
// memory; every spin has an iteration limit, after which the CTA raises STRADS_STATUS_WAIT_EXPIRED
// and leaves (the launch is cooperative, so all CTAs are resident and the limit is never met in practice).
// The kept list equals that of the full-Gram walk: same correlations (sparse_dot), same order.
#include "strads_internal.cuh"

namespace strads {
namespace {

constexpr int kThreads = 256;
constexpr int kBatch = 32;
constexpr int kStage = 1024;          // entries of a column staged in shared memory (longer columns: global)
constexpr unsigned int kSpinLimit = 1u << 26;

// Grid-wide barrier.  Returns false when the wait gave up (or an earlier one did).
__device__ bool grid_barrier(WalkControl* c, unsigned int n_ctas, unsigned int* status) {
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
      while (*gen == g && ++it < kSpinLimit) {}
      if (*gen == g) { ok = false; atomicOr(status, STRADS_STATUS_WAIT_EXPIRED); c->failed = 1; }
    }
    __threadfence();
    if (*reinterpret_cast<volatile int*>(&c->failed)) ok = false;
    s_ok = ok;
  }
  __syncthreads();
  return s_ok != 0;
}

__global__ void __launch_bounds__(kThreads) k_walk_csc(Problem p, const int* __restrict__ cand, int n_cand,
                                                        int only_if_short, int* __restrict__ kept_out) {
  if (only_if_short && !p.st->window_short) return;      // uniform over the grid: nobody reaches a barrier
  __shared__ int arow[kStage];
  __shared__ float aval[kStage];
  __shared__ int s_pos[kBatch];
  __shared__ unsigned int s_keep;
  WalkControl* c = p.walk_ctl;
  const int W = p.mask_words;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned int n_ctas = gridDim.x;
  unsigned int* blocked = p.walk_blocked;
  unsigned int* rows = p.walk_rows;
  const double rho = (double)p.rho;

  if (blockIdx.x == 0) {
    for (int w = tid; w < W; w += kThreads) blocked[w] = 0u;
    if (tid == 0) { c->m = 0; c->cursor = 0; c->n_kept = 0; c->examined = 0; c->done = 0; }
  }
  bool ok = grid_barrier(c, n_ctas, &p.st->status);

  while (ok) {
    // ---- A: CTA 0, warp 0: the next <= 32 candidates at or after the cursor that are not blocked ----
    if (blockIdx.x == 0 && tid < 32) {
      int m = 0;
      int cur = c->cursor;
      while (cur < n_cand && m < kBatch) {
        const int wbase = (cur >> 5) + lane;
        unsigned int freew = 0u;
        if (wbase < W) {
          freew = ~__ldcg(&blocked[wbase]);
          const int first = wbase << 5;
          if (first < cur) freew &= 0xffffffffu << (cur - first);
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
        int slot = m + incl - cnt;
        unsigned int fw = freew;
        while (fw && slot < kBatch) {
          const int b = __ffs(fw) - 1;
          fw &= fw - 1;
          const int ps = (wbase << 5) + b;
          c->pos[slot] = ps;
          c->cval[slot] = cand[ps];
          ++slot;
        }
        m = min(kBatch, m + total);
        if (m < kBatch) cur = ((cur >> 5) + 32) << 5;
      }
      if (lane == 0) c->m = m;
    }
    ok = grid_barrier(c, n_ctas, &p.st->status);
    if (!ok) break;
    const int m = *reinterpret_cast<volatile int*>(&c->m);
    if (m == 0) {                                          // list exhausted
      if (blockIdx.x == 0 && tid == 0) c->examined = n_cand;
      break;
    }
    if (tid < kBatch) s_pos[tid] = __ldcg(&c->pos[min(tid, m - 1)]);
    __syncthreads();

    // ---- B: all CTAs: conflict rows of the batch.  CTA k works on batch member k mod m. ----
    {
      const int q = blockIdx.x % m;
      const int share = (int)((n_ctas - q + m - 1) / m);   // CTAs working on member q
      const int mine = blockIdx.x / m;                      // this CTA's rank among them
      const int a = s_pos[q];
      const int ja = cand[a];
      const long long a0 = p.xptr[ja];
      const int na = (int)(p.xptr[ja + 1] - a0);
      const bool staged = na <= kStage;
      if (staged)
        for (int e = tid; e < na; e += kThreads) { arow[e] = p.xrow[a0 + e]; aval[e] = p.xv[a0 + e]; }
      __syncthreads();
      const int* ar = staged ? arow : p.xrow + a0;
      const float* av = staged ? aval : p.xv + a0;
      const double n2a = p.n2[ja];
      for (int w = (a >> 5) + mine * (kThreads / 32) + warp; w < W; w += share * (kThreads / 32)) {
        const int b = w * 32 + lane;
        bool hit = false;
        if (b < n_cand && b != a) {
          const int jb = cand[b];
          const float dot = sparse_dot(ar, av, na, p, jb);
          const double den = sqrt(n2a * p.n2[jb]);
          hit = den > 0.0 && fabs((double)dot) >= rho * den;
        }
        const unsigned int word = __ballot_sync(0xffffffffu, hit);
        if (lane == 0) rows[(long long)q * W + w] = word;
      }
    }
    ok = grid_barrier(c, n_ctas, &p.st->status);
    if (!ok) break;

    // ---- C: CTA 0 decides the batch in order and extends the mask ----
    if (blockIdx.x == 0) {
      if (tid < 32) {
        const unsigned int valid = m >= 32 ? 0xffffffffu : ((1u << m) - 1u);
        const long long my_row = (long long)min(lane, m - 1) * W;
        unsigned int confl = 0u;
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
          const int pb = s_pos[b];                       // (entries past m repeat the last member; masked below)
          confl |= ((__ldcg(&rows[my_row + (pb >> 5)]) >> (pb & 31)) & 1u) << b;
        }
        confl &= valid & ~((2u << lane) - 1u);           // later members only; a row is valid from its own word on
        if (lane >= m) confl = 0u;
        unsigned int cq[kBatch];
#pragma unroll
        for (int q = 0; q < kBatch; ++q) cq[q] = __shfl_sync(0xffffffffu, confl, q);
        unsigned int alive = valid, keep = 0u;
#pragma unroll
        for (int q = 0; q < kBatch; ++q)
          if ((alive >> q) & 1u) { keep |= 1u << q; alive &= ~cq[q]; }
        const int nk = c->n_kept;
        const int room = p.n_keep - nk;
        bool full = false;
        if (__popc(keep) >= room) {
          while (__popc(keep) > room) keep &= ~(1u << (31 - __clz(keep)));
          full = true;
        }
        if ((keep >> lane) & 1u) kept_out[nk + __popc(keep & ((1u << lane) - 1u))] = __ldcg(&c->cval[lane]);
        if (lane == 0) {
          s_keep = keep;
          c->n_kept = nk + __popc(keep);
          if (full) { c->examined = s_pos[31 - __clz(keep)] + 1; c->done = 1; }
          else c->cursor = s_pos[m - 1] + 1;
        }
      }
      __syncthreads();
      const unsigned int keep = s_keep;
      for (int w = tid; w < W; w += kThreads) {
        unsigned int acc = 0u;
        unsigned int k = keep;
        while (k) {
          const int q = __ffs(k) - 1;
          k &= k - 1;
          if (w >= (s_pos[q] >> 5)) acc |= __ldcg(&rows[(long long)q * W + w]);
        }
        if (acc) blocked[w] |= acc;
      }
    }
    ok = grid_barrier(c, n_ctas, &p.st->status);
    if (!ok) break;
    if (*reinterpret_cast<volatile int*>(&c->done)) break;
  }

  if (blockIdx.x == 0) {
    __syncthreads();
    const int nk = *reinterpret_cast<volatile int*>(&c->n_kept);
    for (int i = nk + tid; i < p.n_keep; i += kThreads) kept_out[i] = -1;
    if (tid == 0) {
      p.st->counts[1] = c->examined; p.st->counts[2] = nk; p.st->counts[3] = 0;
      p.st->amb_count = 0; p.st->window_short = 0; p.st->prefer_walk = 1;
      c->failed = 0;
    }
  }
}

}  // namespace

// Largest cooperative grid (at most 2 CTAs per SM) for this device.
cudaError_t prepare_walk_csc(const Problem& p, int* grid_out) {
  int per_sm = 0;
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_walk_csc, kThreads, 0);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  *grid_out = p.sm_count * (per_sm < 2 ? per_sm : 2);
  return cudaSuccess;
}

cudaError_t launch_walk_csc(const Problem& p, const int* cand, int n_cand, int grid, bool only_if_short, int* kept_out,
                            cudaStream_t s) {
  Problem q = p;
  int ois = only_if_short ? 1 : 0;
  void* args[] = {&q, &cand, &n_cand, &ois, &kept_out};
  return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(k_walk_csc), dim3(grid), dim3(kThreads), args, 0, s);
}

}  // namespace strads
