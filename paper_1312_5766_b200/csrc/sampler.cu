// SAP step 1 / Algorithm 1 "draw a set U of P' coefficients from p(j)": priority sampling without
// replacement, p(j) ~ delta_j^2 + eta (Theorem 1's weight with Algorithm 1's floor eta).
//
// Every coefficient gets the race key (bits of T_j) << 32 | j, T_j = E_j / w_j with E_j a unit
// exponential made from the Philox4x32-10 word of (seed, t, j).  The P' smallest keys, in ascending
// order, are the candidates.  They are found by a multi-CTA radix select that recomputes the keys in
// every pass instead of storing them (one read of delta[J] per pass, no 8J-byte key array):
//
//   k_sample_hist    pass 1: histogram of the top 12 key bits; the last CTA to finish scans it and
//                    publishes the boundary bin (all keys below it are winners, the bin itself holds
//                    the rest).  For an exponential race the boundary bin holds < ~0.1 P' keys in
//                    expectation whatever the weights are; if it ever exceeds the boundary buffer,
//                    that CTA alone refines the boundary over further 12-bit digits (rare, exact).
//   k_sample_collect pass 2: a "sure" key goes to the group of its histogram bin in the `sure` buffer (group
//                    offsets from the first pass's counts), a "boundary" key to the boundary buffer.
//   k_sample_rank_bins  (the default) orders the winners: bins are in key order already, so every key is
//                    ranked inside its own group only, and the boundary keys among themselves.
//   k_sample_patch   corrects a list drawn one round ahead for the coefficients the last update changed.
//   k_sample_rank_direct (P' <= 2048) / k_sample_sort_chunks + k_sample_rank (larger P'): ordering without
//                    group arrays (counting over the whole buffer; 1024-key chunk sorts in shared memory,
//                    then ranks by binary search in the other chunks); used by strads_sample_static.
#include <cstddef>
#include <mutex>

#include "strads_internal.cuh"

namespace strads {

namespace {

constexpr int kThreads = 256;

// Whether the race key of a coefficient (last change d, Philox word x) is certainly above `cut` (> 0), from
// a few operations instead of the whole key: T = E / w and the computed E is never below
// v = (x + 1/2) / 2^32 (-ln(1 - v) >= v; checked against the key's arithmetic over its whole range of x), so
// v > 1.01 cut w  implies  T > cut.  Nearly all coefficients are far above the boundary of the P' smallest.
__device__ __forceinline__ bool key_surely_above(float cut, float d, float eta, uint32_t x, int mode) {
  const float w = priority_weight(d, eta, mode);
  const float v = __fmaf_rn(__uint2float_rn(x), __uint_as_float(0x2f800000u), __uint_as_float(0x2f000000u));
  return v > __fmul_rn(__fmul_rn(cut, w), 1.01f);
}

// Calls f(key) for each of the (up to) four coefficients of Philox block g, leaving out those whose key is
// certainly above `cut` (cut <= 0: none is left out).
template <typename F>
__device__ __forceinline__ void for_keys_of_group(const Problem& p, unsigned long long t, long long g, float cut, F&& f) {
  uint32_t w[4];
  philox4x32_10((uint32_t)g, (uint32_t)t, (uint32_t)(t >> 32), 0u, (uint32_t)p.seed, (uint32_t)(p.seed >> 32), w);
  const long long j0 = g * 4;
  const int mode = weight_mode_of(p.flags);
  if (cut > 0.f && p.part_count <= 1 && j0 + 3 < p.J) {
    const float4 d = __ldg(reinterpret_cast<const float4*>(p.delta + j0));
    if (!key_surely_above(cut, d.x, p.eta, w[0], mode)) f(race_key64(d.x, p.eta, w[0], (uint32_t)j0, mode));
    if (!key_surely_above(cut, d.y, p.eta, w[1], mode)) f(race_key64(d.y, p.eta, w[1], (uint32_t)j0 + 1, mode));
    if (!key_surely_above(cut, d.z, p.eta, w[2], mode)) f(race_key64(d.z, p.eta, w[2], (uint32_t)j0 + 2, mode));
    if (!key_surely_above(cut, d.w, p.eta, w[3], mode)) f(race_key64(d.w, p.eta, w[3], (uint32_t)j0 + 3, mode));
    return;
  }
  if (p.part_count > 1) {                              // only the coefficients this scheduler owns take part
    const unsigned int S = (unsigned)p.part_count, r0 = (unsigned int)j0 % S;
#pragma unroll
    for (unsigned int i = 0; i < 4; ++i)
      if (j0 + i < p.J && (r0 + i) % S == (unsigned)p.part_index) {
        const float d = __ldg(p.delta + j0 + i);
        if (cut > 0.f && key_surely_above(cut, d, p.eta, w[i], mode)) continue;
        f(race_key64(d, p.eta, w[i], (uint32_t)(j0 + i), mode));
      }
    return;
  }
  if (j0 + 3 < p.J) {
    const float4 d = __ldg(reinterpret_cast<const float4*>(p.delta + j0));
    f(race_key64(d.x, p.eta, w[0], (uint32_t)j0, mode));
    f(race_key64(d.y, p.eta, w[1], (uint32_t)j0 + 1, mode));
    f(race_key64(d.z, p.eta, w[2], (uint32_t)j0 + 2, mode));
    f(race_key64(d.w, p.eta, w[3], (uint32_t)j0 + 3, mode));
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (j0 + i < p.J) f(race_key64(p.delta[j0 + i], p.eta, w[i], (uint32_t)(j0 + i), mode));
  }
}

// The same with a cutoff, for a whole warp: lane l looks at Philox block g0 + l.  Few coefficients survive the
// cheap test, so computing their keys on the spot would leave most lanes idle while one works; the survivors
// (index, Philox word) go to a queue of the warp in shared memory instead and the keys of a full queue are
// computed by all lanes together.  drain_keys() must follow the last call.
constexpr int kQueue = 256;              // entries per warp; a call appends at most 128
struct KeyQueue { uint2* slots; int n; };

template <typename F>
__device__ __forceinline__ void drain_keys(const Problem& p, KeyQueue& q, F&& f) {
  const int mode = weight_mode_of(p.flags);
  __syncwarp();
  for (int i = (int)(threadIdx.x & 31); i < q.n; i += 32) {
    const uint2 e = q.slots[i];
    f(race_key64(__ldg(p.delta + e.x), p.eta, e.y, e.x, mode));
  }
  __syncwarp();
  q.n = 0;
}

template <typename F>
__device__ __forceinline__ void queue_keys_of_groups(const Problem& p, unsigned long long t, long long g0, long long groups,
                                                     float cut, KeyQueue& q, F&& f) {
  const int lane = threadIdx.x & 31;
  const long long g = g0 + lane;
  const int mode = weight_mode_of(p.flags);
  if (p.part_count <= 1 && (g0 + 32) * 4 <= p.J) {
    // The common case, kept lean because the pass is bound by instruction issue (about 300 instructions per lane
    // and call before, a third of them Philox): one scheduler and all 32 blocks of the warp whole, so no bounds or
    // ownership tests; and since survivors are rare (a fraction of a percent of the coefficients), one vote tells
    // the warp whether there is anything to queue at all -- the four ballots with their ranks run only then.
    uint32_t w[4];
    philox4x32_10((uint32_t)g, (uint32_t)t, (uint32_t)(t >> 32), 0u, (uint32_t)p.seed, (uint32_t)(p.seed >> 32), w);
    const float4 v = __ldg(reinterpret_cast<const float4*>(p.delta) + g);
    const float d[4] = {v.x, v.y, v.z, v.w};
    bool in[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) in[i] = !key_surely_above(cut, d[i], p.eta, w[i], mode);
    if (!__any_sync(0xffffffffu, in[0] | in[1] | in[2] | in[3])) return;
    const uint32_t j0 = (uint32_t)g * 4u;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const unsigned int mask = __ballot_sync(0xffffffffu, in[i]);
      if (in[i]) q.slots[q.n + __popc(mask & ((1u << lane) - 1u))] = make_uint2(j0 + i, w[i]);
      q.n += __popc(mask);
    }
    if (q.n > kQueue - 128) drain_keys(p, q, f);
    return;
  }
  uint32_t w[4] = {0u, 0u, 0u, 0u};
  float d[4] = {0.f, 0.f, 0.f, 0.f};
  const long long j0 = g * 4;
  if (g < groups) {
    philox4x32_10((uint32_t)g, (uint32_t)t, (uint32_t)(t >> 32), 0u, (uint32_t)p.seed, (uint32_t)(p.seed >> 32), w);
    if (j0 + 3 < p.J) {
      const float4 v = __ldg(reinterpret_cast<const float4*>(p.delta + j0));
      d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) if (j0 + i < p.J) d[i] = p.delta[j0 + i];
    }
  }
  const unsigned int S = (unsigned)max(p.part_count, 1), r0 = (unsigned int)j0 % S;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const bool in = g < groups && j0 + i < p.J && (S == 1u || (r0 + i) % S == (unsigned)p.part_index) &&
                    !key_surely_above(cut, d[i], p.eta, w[i], mode);
    const unsigned int mask = __ballot_sync(0xffffffffu, in);
    if (in) q.slots[q.n + __popc(mask & ((1u << lane) - 1u))] = make_uint2((uint32_t)(j0 + i), w[i]);
    q.n += __popc(mask);
  }
  if (q.n > kQueue - 128) drain_keys(p, q, f);
}

// Whole CTA (kThreads threads): the bin b with before(b) < k_rem <= before(b) + h[b], where before(b)
// is the number of keys in bins below b.  Exactly one thread finds it and writes *bin / *before.
__device__ void find_bin(const unsigned int* h, int nbins, long long k_rem, int* bin, long long* before) {
  __shared__ long long warp_tot[kThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int per = (nbins + kThreads - 1) / kThreads;
  const int b0 = tid * per;
  long long mine = 0;
  for (int b = b0; b < b0 + per && b < nbins; ++b) mine += h[b];
  long long incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const long long v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) warp_tot[wid] = incl;
  __syncthreads();
  long long base = 0;
  for (int w = 0; w < wid; ++w) base += warp_tot[w];
  incl += base;
  const long long excl = incl - mine;
  if (excl < k_rem && k_rem <= incl) {
    long long cum = excl;
    int b = b0;
    for (; b < b0 + per - 1 && b < nbins - 1; ++b) {
      if (cum + h[b] >= k_rem) break;
      cum += h[b];
    }
    *bin = b;
    *before = cum;
  }
  __syncthreads();
}

// mode 0: plain.  mode 1: bins only the keys below a cutoff carried over from the previous round (four times that
// round's boundary; the keys certainly above it are not even computed); if fewer than P' keys turn out to lie
// below it, the last CTA redoes the pass in full by itself.
__global__ void __launch_bounds__(kThreads, 4) k_sample_hist(Problem p, int mode) {
  chain_begin();
  __shared__ unsigned int sh[kHistBins];
  __shared__ int s_last;
  __shared__ SelectState s_sel;
  const int tid = threadIdx.x;
  for (int b = tid; b < kHistBins; b += kThreads) sh[b] = 0;
  __syncthreads();
  const unsigned long long t = *p.round_ptr + (unsigned long long)p.round_ahead;
  const long long groups = (p.J + 3) >> 2;
  const float cut = mode == 1 ? p.st->t_cut : 0.f;
  const unsigned int cut_bin = cut > 0.f ? (__float_as_uint(cut) >> (32 - kHistBits)) : (unsigned)kHistBins;   // bins below it are complete
  // Guided pass: the keys below the cutoff (a few times P' of them) are also saved, so that the collect pass can
  // take the winners from those instead of going through all J coefficients again.
  const bool save = cut > 0.f && p.survivors != nullptr;
  auto count = [&](unsigned long long key) {
    const unsigned int bin = (unsigned int)(key >> (64 - kHistBits));
    if (bin < cut_bin) {
      atomicAdd(&sh[bin], 1u);
      if (save) {
        const unsigned int at = atomicAdd(&p.st->surv_count, 1u);
        if (at < (unsigned)p.cap_survivors) p.survivors[at] = key;
      }
    }
  };
  if (cut > 0.f) {
    __shared__ uint2 s_queue[kThreads / 32][kQueue];
    KeyQueue q = {s_queue[tid >> 5], 0};
    for (long long g0 = (long long)blockIdx.x * kThreads + (tid & ~31); g0 < groups; g0 += (long long)gridDim.x * kThreads)
      queue_keys_of_groups(p, t, g0, groups, cut, q, count);
    drain_keys(p, q, count);
  } else {
    for (long long g = (long long)blockIdx.x * kThreads + tid; g < groups; g += (long long)gridDim.x * kThreads)
      for_keys_of_group(p, t, g, 0.f, count);
  }
  __syncthreads();
  for (int b = tid; b < kHistBins; b += kThreads)
    if (sh[b]) atomicAdd(&p.hist[b], sh[b]);
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&p.st->hist_ticket, 1u) == gridDim.x - 1);
  __syncthreads();
  if (!s_last) return;

  // ---- last CTA: every other CTA's histogram is visible now ----
  __threadfence();
  {
    // all loads first, then the stores (a store between two loads would order them: one round trip per bin)
    unsigned int v[kHistBins / kThreads];
#pragma unroll
    for (int u = 0; u < kHistBins / kThreads; ++u) v[u] = __ldcg(&p.hist[tid + u * kThreads]);
#pragma unroll
    for (int u = 0; u < kHistBins / kThreads; ++u) {
      sh[tid + u * kThreads] = v[u];
      p.hist[tid + u * kThreads] = 0;                 // ready for the next round
    }
  }
  __syncthreads();
  __shared__ int s_bin;
  __shared__ long long s_before;
  bool solo = false;
  if (cut > 0.f) {                                     // enough keys below the cutoff?
    __shared__ unsigned int s_total;
    if (tid == 0) s_total = 0u;
    __syncthreads();
    unsigned int mine = 0u;
    for (int b = tid; b < kHistBins; b += kThreads) mine += sh[b];
    atomicAdd(&s_total, mine);
    __syncthreads();
    if (s_total < (unsigned)p.n_cand) {
      // The guide was too low (the weights collapsed since the last round: the end of the first sweep, say).  Rare,
      // so this CTA redoes the pass alone and in full rather than the whole grid being launched a second time every
      // round just in case: some milliseconds once, for 10^7 coefficients.
      solo = true;
      __syncthreads();
      for (int b = tid; b < kHistBins; b += kThreads) sh[b] = 0;
      __syncthreads();
      for (long long g = tid; g < groups; g += kThreads)
        for_keys_of_group(p, t, g, 0.f, [&](unsigned long long key) { atomicAdd(&sh[(unsigned int)(key >> (64 - kHistBits))], 1u); });
      __syncthreads();
    }
  }
  find_bin(sh, kHistBins, p.n_cand, &s_bin, &s_before);
  if (tid == 0) {
    // (every CTA's appends are done and visible: they precede its ticket)
    p.st->surv_valid = (save && !solo && __ldcg(&p.st->surv_count) <= (unsigned)p.cap_survivors) ? 1 : 0;
    p.st->sample_redo = 0;
    // next round's cutoff: four times the upper edge of this boundary bin (none if that is not a finite number)
    const unsigned int edge = ((unsigned int)s_bin + 1u) << (32 - kHistBits);
    p.st->t_cut = edge < 0x7f800000u ? __fmul_rn(4.0f, __uint_as_float(edge)) : 0.f;
    p.st->hist_ticket = 0;
    p.st->sure_count = 0;                             // append cursors of the collect pass that follows
    p.st->boundary_count = 0;
    s_sel.prefix = (unsigned long long)s_bin;
    s_sel.bits = kHistBits;
    s_sel.n_sure = (int)s_before;
    s_sel.n_boundary = (int)sh[s_bin];
  }
  __syncthreads();
  if (p.bin_off != nullptr) {
    // Where the sure keys of every bin below the boundary bin start in the `sure` buffer (exclusive prefix of the
    // counts; the boundary bin's own sure keys, if it gets refined, follow at s_before), and the bins' cursors:
    // the collect pass then leaves the winners grouped by their top 12 bits, and ordering them is a matter of
    // ranking every key inside its own small group.
    __shared__ unsigned int s_wtot[kThreads / 32];
    constexpr int kPer = kHistBins / kThreads;
    const int b0 = tid * kPer, lane = tid & 31, wid = tid >> 5;
    unsigned int mine = 0u;
#pragma unroll
    for (int u = 0; u < kPer; ++u) mine += (b0 + u < s_bin) ? sh[b0 + u] : 0u;
    unsigned int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) s_wtot[wid] = incl;
    __syncthreads();
    unsigned int run = incl - mine;
    for (int w = 0; w < wid; ++w) run += s_wtot[w];
#pragma unroll
    for (int u = 0; u < kPer; ++u) {                   // counts -> offsets in place (nobody needs the counts any more)
      const unsigned int c = (b0 + u < s_bin) ? sh[b0 + u] : 0u;
      sh[b0 + u] = run;
      run += c;
    }
    if (tid == kThreads - 1) p.bin_off[kHistBins] = (int)run;
    __syncthreads();
    for (int b = tid; b < kHistBins; b += kThreads) {  // coalesced
      p.bin_off[b] = (int)sh[b];
      p.bin_cur[b] = 0u;
    }
    __syncthreads();
  }
  // Rare: the boundary bin does not fit the buffer -> refine digit by digit with this CTA alone.
  while (s_sel.n_boundary > p.cap_boundary && s_sel.bits < 64) {
    const int bits = s_sel.bits;
    const int width = min(kHistBits, 64 - bits);
    const unsigned long long prefix = s_sel.prefix;
    __syncthreads();
    for (int b = tid; b < kHistBins; b += kThreads) sh[b] = 0;
    __syncthreads();
    for (long long g = tid; g < groups; g += kThreads)
      for_keys_of_group(p, t, g, 0.f, [&](unsigned long long key) {
        if ((key >> (64 - bits)) == prefix)
          atomicAdd(&sh[(key >> (64 - bits - width)) & ((1u << width) - 1u)], 1u);
      });
    __syncthreads();
    find_bin(sh, 1 << width, (long long)p.n_cand - s_sel.n_sure, &s_bin, &s_before);
    if (tid == 0) {
      s_sel.prefix = (prefix << width) | (unsigned long long)s_bin;
      s_sel.bits = bits + width;
      s_sel.n_sure += (int)s_before;
      s_sel.n_boundary = (int)sh[s_bin];
      atomicOr(&p.st->status, STRADS_STATUS_SAMPLER_REFINED);
    }
    __syncthreads();
  }
  if (tid == 0) p.st->sel = s_sel;
}

__global__ void __launch_bounds__(kThreads) k_sample_collect(Problem p) {
  chain_begin();
  const SelectState sel = p.st->sel;
  const unsigned long long t = *p.round_ptr + (unsigned long long)p.round_ahead;
  const long long groups = (p.J + 3) >> 2;
  const int shift = 64 - sel.bits;
  // keys certainly above the boundary's upper edge are not computed
  unsigned long long edge = sel.bits <= 32 ? ((sel.prefix + 1ull) << (32 - sel.bits)) : (sel.prefix >> (sel.bits - 32));
  const float cut = edge < 0x7f800000ull && edge > 0ull ? __uint_as_float((unsigned int)edge) : 0.f;
  const unsigned int top_bin = (unsigned int)(sel.prefix >> (sel.bits - kHistBits));   // the boundary bin of the first pass
  auto take = [&](unsigned long long key) {
    const unsigned long long pfx = key >> shift;
    if (pfx < sel.prefix) {
      unsigned int i;
      if (p.bin_off != nullptr) {                      // into the group of its histogram bin
        const unsigned int bin = min((unsigned int)(key >> (64 - kHistBits)), top_bin);
        i = (unsigned int)p.bin_off[bin] + atomicAdd(&p.bin_cur[bin], 1u);
      } else {
        i = atomicAdd(&p.st->sure_count, 1u);
      }
      if (i < (unsigned)p.cap_sure) p.sure[i] = key;
    } else if (pfx == sel.prefix) {
      const unsigned int i = atomicAdd(&p.st->boundary_count, 1u);
      if (i < (unsigned)p.cap_boundary) p.boundary[i] = key;
    }
  };
  const int tid = threadIdx.x;
  if (p.st->surv_valid) {                              // every key below the first pass's cutoff is at hand
    const unsigned int n = p.st->surv_count;
    for (unsigned int i = blockIdx.x * (unsigned)kThreads + tid; i < n; i += gridDim.x * (unsigned)kThreads)
      take(__ldcg(p.survivors + i));
    return;
  }
  if (cut > 0.f) {
    __shared__ uint2 s_queue[kThreads / 32][kQueue];
    KeyQueue q = {s_queue[tid >> 5], 0};
    for (long long g0 = (long long)blockIdx.x * kThreads + (tid & ~31); g0 < groups; g0 += (long long)gridDim.x * kThreads)
      queue_keys_of_groups(p, t, g0, groups, cut, q, take);
    drain_keys(p, q, take);
  } else {
    for (long long g = (long long)blockIdx.x * kThreads + tid; g < groups; g += (long long)gridDim.x * kThreads)
      for_keys_of_group(p, t, g, 0.f, take);
  }
}

// Ascending bitonic sort of n (a power of two) keys in shared memory by the whole CTA.
__device__ void bitonic_sort(unsigned long long* a, int n) {
  for (int k = 2; k <= n; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = threadIdx.x; i < (n >> 1); i += blockDim.x) {
        const int lo = ((i & ~(j - 1)) << 1) | (i & (j - 1));
        const int hi = lo | j;
        const unsigned long long x = a[lo], y = a[hi];
        const bool up = (lo & k) == 0;
        if ((x > y) == up) { a[lo] = y; a[hi] = x; }
      }
      __syncthreads();
    }
  }
}

__device__ int pow2_ceil(int n) { int v = 1; while (v < n) v <<= 1; return v; }

constexpr int kChunk = 1024;             // keys sorted by one CTA

// Which slice of which buffer CTA `c` owns: sure chunks first, then boundary chunks.
struct ChunkRef { unsigned long long* base; int n; int first; bool is_sure; };
__device__ __forceinline__ ChunkRef chunk_of(const Problem& p, const SelectState& sel, int c) {
  const int n_sure = min(sel.n_sure, p.cap_sure), n_bnd = min(sel.n_boundary, p.cap_boundary);
  const int sure_chunks = (p.cap_sure + kChunk - 1) / kChunk;
  ChunkRef r;
  r.is_sure = c < sure_chunks;
  const int ci = r.is_sure ? c : c - sure_chunks;
  const int total = r.is_sure ? n_sure : n_bnd;
  r.first = ci * kChunk;
  r.n = max(0, min(kChunk, total - r.first));
  r.base = (r.is_sure ? p.sure : p.boundary) + r.first;
  return r;
}

// Step 1 of the final ordering: every CTA sorts one chunk of up to 1024 collected keys in shared memory
// (bitonic) and writes it back in place.  One CTA sorting all P' keys would be bound by its own shared-memory
// bandwidth (~100 us for 16,384 keys); chunks run on as many SMs as there are chunks.
__global__ void __launch_bounds__(512) k_sample_sort_chunks(Problem p) {
  chain_begin();
  __shared__ unsigned long long keys[kChunk];
  const SelectState sel = p.st->sel;
  const ChunkRef ch = chunk_of(p, sel, blockIdx.x);
  if (ch.n == 0) return;
  const int n = pow2_ceil(ch.n);
  for (int i = threadIdx.x; i < n; i += blockDim.x) keys[i] = i < ch.n ? ch.base[i] : ~0ull;
  __syncthreads();
  bitonic_sort(keys, n);
  for (int i = threadIdx.x; i < ch.n; i += blockDim.x) ch.base[i] = keys[i];
}

// Number of keys < key in a sorted array (keys are distinct).
__device__ __forceinline__ int count_less(const unsigned long long* a, int n, unsigned long long key) {
  int lo = 0, hi = n;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (a[mid] < key) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// Step 2: the rank of a key among all collected keys = its index in its own chunk + the number of smaller
// keys in every other chunk of its buffer (+ n_sure for boundary keys: every sure key is smaller).  The key
// of rank r < P' is candidate r.  Each other chunk is staged in shared memory and searched there.
__global__ void __launch_bounds__(512) k_sample_rank(Problem p, int* cand_out) {
  chain_begin();
  __shared__ unsigned long long other[kChunk];
  const SelectState sel = p.st->sel;
  const ChunkRef ch = chunk_of(p, sel, blockIdx.x);
  if (blockIdx.x == 0 && threadIdx.x == 0) { p.st->counts[0] = p.n_cand; p.st->surv_count = 0; }
  if (ch.n == 0) return;
  const int n_sure = min(sel.n_sure, p.cap_sure), n_bnd = min(sel.n_boundary, p.cap_boundary);
  const unsigned long long* buf = ch.is_sure ? p.sure : p.boundary;
  const int total = ch.is_sure ? n_sure : n_bnd;
  const int i0 = threadIdx.x, i1 = threadIdx.x + 512;           // this thread's (up to) two keys
  const unsigned long long k0 = i0 < ch.n ? __ldcg(ch.base + i0) : 0ull, k1 = i1 < ch.n ? __ldcg(ch.base + i1) : 0ull;
  int r0 = i0 + (ch.is_sure ? 0 : n_sure), r1 = i1 + (ch.is_sure ? 0 : n_sure);
  for (int o = 0; o < total; o += kChunk) {
    if (o == ch.first) continue;
    const int n = min(kChunk, total - o);
    __syncthreads();
    for (int e = threadIdx.x; e < n; e += 512) other[e] = __ldcg(buf + o + e);
    __syncthreads();
    r0 += count_less(other, n, k0);
    r1 += count_less(other, n, k1);
  }
  if (i0 < ch.n && r0 < p.n_cand) { cand_out[r0] = (int)(k0 & 0xffffffffull); if (p.keys_out) p.keys_out[r0] = k0; }
  if (i1 < ch.n && r1 < p.n_cand) { cand_out[r1] = (int)(k1 & 0xffffffffull); if (p.keys_out) p.keys_out[r1] = k1; }
}

// Small P': the order of the winners straight from the definition, with no sort.  The rank of a key is the
// number of smaller keys in its buffer (+ n_sure for boundary keys: every sure key is smaller); the key of
// rank r < P' is candidate r.  A CTA takes 32 keys of one buffer, stages the whole buffer (<= 2048 keys) in
// shared memory and counts with eight threads per key, each over an eighth of the buffer.
constexpr int kDirectMax = 2048;         // P' and the boundary buffer up to this many keys (beyond, sorting is as fast)
constexpr int kDirectKeys = 32;          // keys per CTA
__global__ void __launch_bounds__(256) k_sample_rank_direct(Problem p, int* cand_out) {
  chain_begin();
  __shared__ unsigned long long all[kDirectMax];
  const SelectState sel = p.st->sel;
  if (blockIdx.x == 0 && threadIdx.x == 0) { p.st->counts[0] = p.n_cand; p.st->surv_count = 0; }
  const int n_sure = min(sel.n_sure, p.cap_sure), n_bnd = min(sel.n_boundary, p.cap_boundary);
  const int sure_ctas = (p.cap_sure + kDirectKeys - 1) / kDirectKeys;
  const bool is_sure = (int)blockIdx.x < sure_ctas;
  const int first = (is_sure ? blockIdx.x : blockIdx.x - sure_ctas) * kDirectKeys;
  const int total = is_sure ? n_sure : n_bnd;
  if (first >= total) return;
  const unsigned long long* buf = is_sure ? p.sure : p.boundary;
  for (int i = threadIdx.x; i < total; i += 256) all[i] = __ldcg(buf + i);
  __syncthreads();
  const int k = first + (threadIdx.x >> 3), slice = threadIdx.x & 7;
  const unsigned long long key = k < total ? all[k] : 0ull;
  int below = 0;                                        // thread `slice` looks at keys slice, slice + 8, ...: the eight
#pragma unroll 8                                        // threads of a key read eight consecutive words (no bank conflict)
  for (int i = slice; i < total; i += 8) below += all[i] < key;
  below += __shfl_xor_sync(0xffffffffu, below, 1);
  below += __shfl_xor_sync(0xffffffffu, below, 2);
  below += __shfl_xor_sync(0xffffffffu, below, 4);
  const int rank = below + (is_sure ? 0 : n_sure);
  if (slice == 0 && k < total && rank < p.n_cand) {
    cand_out[rank] = (int)(key & 0xffffffffull);
    if (p.keys_out) p.keys_out[rank] = key;
  }
}

// Ordering the winners when the collect pass grouped them by histogram bin (bin_off): bins are in key order, so a
// sure key's rank is the start of its bin's group plus the number of smaller keys inside the group -- a few
// hundred keys (an exponential race spreads the winners over dozens of bins, at most ~P' / 16 in one) -- and a
// boundary key's is n_sure plus the number of smaller boundary keys.  Eight threads per key, all in one kernel.
__global__ void __launch_bounds__(256) k_sample_rank_bins(Problem p, int* cand_out) {
  chain_begin();
  const SelectState sel = p.st->sel;
  if (blockIdx.x == 0 && threadIdx.x == 0) { p.st->counts[0] = p.n_cand; p.st->surv_count = 0; }
  const int n_sure = min(sel.n_sure, p.cap_sure), n_bnd = min(sel.n_boundary, p.cap_boundary);
  const int i = (blockIdx.x * 256 + threadIdx.x) >> 3, slice = threadIdx.x & 7;    // eight threads per key
  const unsigned long long* buf = p.sure;
  unsigned long long key = 0ull;
  int first = 0, count = 0, base = 0;
  if (i < n_sure) {
    const int top_bin = (int)(sel.prefix >> (sel.bits - kHistBits));
    key = p.sure[i];
    const int bin = min((int)(key >> (64 - kHistBits)), top_bin);
    first = p.bin_off[bin];
    count = (bin < top_bin ? p.bin_off[bin + 1] : n_sure) - first;
    base = first;
  } else if (i - n_sure < n_bnd) {
    key = p.boundary[i - n_sure];
    count = n_bnd; buf = p.boundary; base = n_sure;
  }
  // thread `slice` looks at keys slice, slice + 8, ... of the group: the eight threads read 64 consecutive bytes.
  // Sixteen loads are under way per thread: the largest groups hold ~P' / 12 keys, and with four loads per trip the
  // threads of those groups made 40 trips of one L2 latency each (18 us for P' = 16,384).
  constexpr int kInFlight = 16;
  int below = 0;
  for (int j = slice; j < count; j += 8 * kInFlight) {
    unsigned long long other[kInFlight];
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) other[u] = j + 8 * u < count ? buf[first + j + 8 * u] : ~0ull;
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) below += other[u] < key ? 1 : 0;
  }
  below += __shfl_xor_sync(0xffffffffu, below, 1);
  below += __shfl_xor_sync(0xffffffffu, below, 2);
  below += __shfl_xor_sync(0xffffffffu, below, 4);
  const int rank = base + below;
  if (slice == 0 && count > 0 && rank < p.n_cand) {
    cand_out[rank] = (int)(key & 0xffffffffull);
    if (p.keys_out) p.keys_out[rank] = key;
  }
}

// Sampling ahead.  The draw of round t is made during round t - 1 (beside its Gram and walk) from the delta of
// that round's start, for P' + P winners instead of P'; the update of round t - 1 then changes delta for at most P
// coefficients.  Every other coefficient keeps its key, and one of them that belongs to the true P' smallest has
// fewer than P' + P keys below it in the early ranking, so it is on the early list L.  The candidates are
// therefore the P' smallest of (L without the updated coefficients) + (the updated coefficients with their new
// keys): exactly the list a draw made now would give.  Rank of an element of L at index i:
// i - #(old keys of updated coefficients below it) + #(new keys below it); of a new key: its insertion point in L
// instead of i.  (An old key below an element of L is itself on L, L being a prefix of the full ranking; a new key
// beyond the end of a list shorter than J ranks >= P' and is left out.)  The <= P old and new keys were left by the
// update (patch_keys); every CTA holds them in shared memory and counts against them by brute force.
// from_cand: the keys are taken from those the pack kernel formed for every candidate (by position in the list), so
// that the correction can run beside the update of the same round instead of behind it.  gate: as for the update
// (0 always; 1 / 2: only the copy on the branch that DeviceState::route names).
__global__ void __launch_bounds__(256) k_sample_patch(Problem p, const unsigned long long* __restrict__ list, int n_list,
                                                      int* __restrict__ cand_out, int from_cand, int gate) {
  chain_begin();
  if (gate != 0 && (p.st->route != 0) != (gate == 2)) return;
  extern __shared__ unsigned long long s_keys[];       // [n_keep] old keys, then [n_keep] new keys
  const int nk = p.st->counts[2];                      // coefficients the update of this round touches
  unsigned long long* old_k = s_keys;
  unsigned long long* new_k = s_keys + p.n_keep;
  for (int a = threadIdx.x; a < nk; a += 256) {
    if (from_cand) {
      const int pos = p.kept_pos[a];
      old_k[a] = p.cand_keys[pos];
      new_k[a] = p.cand_keys[p.n_cand + pos];
    } else {                                           // left by the update, which knew both priorities
      old_k[a] = p.patch_keys[a];
      new_k[a] = p.patch_keys[p.n_keep + a];
    }
  }
  __syncthreads();
  if (blockIdx.x == 0 && threadIdx.x == 0) p.st->counts[0] = p.n_cand;
  const unsigned int full = 0xffffffffu;
  const int list_ctas = (n_list + 31) / 32;            // eight threads per element of the list
  if ((int)blockIdx.x < list_ctas) {
    const int item = (blockIdx.x * 256 + threadIdx.x) >> 3, slice = threadIdx.x & 7;
    const unsigned long long key = item < n_list ? list[item] : 0ull;
    int below_old = 0, below_new = 0, is_old = 0;
    for (int a = slice; a < nk; a += 8) {
      const unsigned long long o = old_k[a];
      below_old += o < key;
      is_old |= o == key;
      below_new += new_k[a] < key;
    }
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
      below_old += __shfl_xor_sync(full, below_old, o);
      below_new += __shfl_xor_sync(full, below_new, o);
      is_old |= __shfl_xor_sync(full, is_old, o);
    }
    if (slice != 0 || item >= n_list || is_old) return;   // (an updated coefficient: its new key stands in for it)
    const int rank = item - below_old + below_new;
    if (rank < p.n_cand) cand_out[rank] = (int)(key & 0xffffffffull);
    return;
  }
  // The CTAs behind them: a warp per new key; its insertion point is counted over the whole list by the 32 lanes
  // (independent, coalesced loads instead of the dependent probes of a binary search).
  const int a = ((int)blockIdx.x - list_ctas) * 8 + (int)(threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (a >= nk) return;
  const unsigned long long key = new_k[a];
  int at = 0, below_old = 0, below_new = 0;
  for (int i = lane; i < n_list; i += 32) at += list[i] < key;
  for (int b = lane; b < nk; b += 32) { below_old += old_k[b] < key; below_new += new_k[b] < key; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    at += __shfl_xor_sync(full, at, o);
    below_old += __shfl_xor_sync(full, below_old, o);
    below_new += __shfl_xor_sync(full, below_new, o);
  }
  if (lane != 0 || (at == n_list && (long long)n_list < p.J)) return;
  const int rank = at - below_old + below_new;
  if (rank < p.n_cand) cand_out[rank] = (int)(key & 0xffffffffull);
}

}  // namespace

// Kernel-wide attribute: the patch kernel's key arrays (sampling ahead is used up to P = 4096: 64 KB).
cudaError_t prepare_sample(const Problem&) {
  return cudaFuncSetAttribute(k_sample_patch, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 8 * 4096);
}

cudaError_t launch_sample_patch(const Problem& p, const Problem& ahead, int* cand_out, cudaStream_t s, bool from_cand,
                                int gate) {
  const int ctas = (ahead.n_cand + 31) / 32 + (p.n_keep + 7) / 8;        // list elements by eight threads, new keys by warp
  return launch_chained(k_sample_patch, ctas, 256, 2 * sizeof(unsigned long long) * (size_t)p.n_keep, s, p,
                        (const unsigned long long*)ahead.keys_out, ahead.n_cand, cand_out, from_cand ? 1 : 0, gate);
}

cudaError_t launch_sample(const Problem& p, int* cand_out, cudaStream_t s) {
  const long long groups = (p.J + 3) >> 2;
  long long blocks = (groups + kThreads - 1) / kThreads;
  // (an early draw runs beside the round's Gram and walk and leaves them most of every SM)
  // otherwise as many CTAs as run at once (four per SM, by the kernels' registers): each pays for its own histogram
  // (cleared, then merged into the global one) once, and the passes are bound by arithmetic, not by the grid's size
  const long long cap = (long long)p.sm_count * (p.round_ahead ? 2 : 4);
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  cudaError_t e;
  // many coefficients: the first pass leaves out the keys far above the last boundary (its last CTA repeats it in
  // full in the rare round where that boundary was a bad guide)
  const bool guided = p.J >= (1 << 19);     // (below that the passes are bound by latency, not by arithmetic)
  if ((e = launch_chained(k_sample_hist, (unsigned)blocks, kThreads, 0, s, p, guided ? 1 : 0)) != cudaSuccess) return e;
  if ((e = launch_chained(k_sample_collect, (unsigned)blocks, kThreads, 0, s, p)) != cudaSuccess) return e;
  if (p.bin_off != nullptr)
    return launch_chained(k_sample_rank_bins, (unsigned)((p.cap_sure + p.cap_boundary + 31) / 32), 256, 0, s, p, cand_out);
  if (p.cap_sure <= kDirectMax && p.cap_boundary <= kDirectMax) {
    const int ctas = (p.cap_sure + kDirectKeys - 1) / kDirectKeys + (p.cap_boundary + kDirectKeys - 1) / kDirectKeys;
    return launch_chained(k_sample_rank_direct, ctas, 256, 0, s, p, cand_out);
  }
  const int chunks = (p.cap_sure + kChunk - 1) / kChunk + (p.cap_boundary + kChunk - 1) / kChunk;
  if ((e = launch_chained(k_sample_sort_chunks, chunks, 512, 0, s, p)) != cudaSuccess) return e;
  return launch_chained(k_sample_rank, chunks, 512, 0, s, p, cand_out);
}

}  // namespace strads

// ------------------------------------------------------------------------------------------------
// strads_sample_static: the same candidate draw for callers that cannot allocate device memory.
//
// The select passes need scratch memory (a 4096-bin histogram, two key buffers, a few counters).
// The handle-based path carves it out of the caller's workspace; here it lives in one file-scope
// device array of fixed size, so a caller that may not call cudaMalloc -- code running inside
// somebody else's memory pool, a plugin whose host forbids allocation after start-up, a real-time
// loop -- still gets the draw.  Every GPU that loads the library holds these ~65 KB until exit.
// ------------------------------------------------------------------------------------------------
namespace strads {
namespace {

struct StaticSampleScratch {
  DeviceState st;
  unsigned int hist[kHistBins];
  unsigned long long sure[STRADS_STATIC_MAX_CANDIDATES];
  unsigned long long boundary[STRADS_STATIC_MAX_CANDIDATES / 2];
};

static __device__ __align__(256) unsigned char g_static_sample_scratch[sizeof(StaticSampleScratch)];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
StaticSampleScratch* g_static_ptr[kMaxDevices] = {};   // device address of the array, per device
int g_static_sms[kMaxDevices] = {};

__global__ void k_static_set_round(StaticSampleScratch* sc, unsigned long long t) { sc->st.round = t; }

}  // namespace
}  // namespace strads

extern "C" int strads_sample_static(const float* delta_dev, int64_t n_cols, float eta, uint64_t seed, uint64_t t,
                                    int32_t n_candidates, uint32_t flags, int32_t* cand_dev, void* stream) {
  using namespace strads;
  if (delta_dev == nullptr || cand_dev == nullptr) return STRADS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(delta_dev) & 15) != 0) return STRADS_ERR_INVALID_ARG;
  if (n_cols < 1 || n_cols >= (1ll << 31) || n_candidates < 1 || n_candidates > n_cols) return STRADS_ERR_INVALID_ARG;
  if (!(eta > 0.f) && !(flags & STRADS_FLAG_UNIFORM_DRAW)) return STRADS_ERR_INVALID_ARG;
  if (n_candidates > STRADS_STATIC_MAX_CANDIDATES) return STRADS_ERR_UNSUPPORTED;   // scratch array is fixed-size

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return STRADS_ERR_CUDA;
  StaticSampleScratch* sc = nullptr;
  int sms = 0;
  {
    // once per device, with that device current: in host code the array's name is only a stand-in,
    // the address a kernel can use comes from cudaGetSymbolAddress
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (g_static_ptr[dev] == nullptr) {
      void* ptr = nullptr;
      if (cudaGetSymbolAddress(&ptr, g_static_sample_scratch) != cudaSuccess || ptr == nullptr) return STRADS_ERR_CUDA;
      if (cudaDeviceGetAttribute(&g_static_sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return STRADS_ERR_CUDA;
      g_static_ptr[dev] = static_cast<StaticSampleScratch*>(ptr);
    }
    sc = g_static_ptr[dev];
    sms = g_static_sms[dev];
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the array keeps whatever the last call left: counters, tickets and histogram must start at zero
  if (cudaMemsetAsync(sc, 0, offsetof(StaticSampleScratch, sure), s) != cudaSuccess) return STRADS_ERR_CUDA;
  k_static_set_round<<<1, 1, 0, s>>>(sc, t);

  Problem p = {};
  p.J = n_cols;
  p.delta = const_cast<float*>(delta_dev);
  p.eta = eta;
  p.seed = seed;
  p.flags = flags;
  p.n_cand = n_candidates;
  p.n_keep = 1;
  p.st = &sc->st;
  p.hist = sc->hist;
  p.sure = sc->sure;
  p.boundary = sc->boundary;
  p.cap_sure = n_candidates;
  p.cap_boundary = STRADS_STATIC_MAX_CANDIDATES / 2;
  p.sm_count = sms;
  p.round_ptr = &sc->st.round;
  return launch_sample(p, cand_dev, s) == cudaSuccess ? STRADS_OK : STRADS_ERR_CUDA;
}
