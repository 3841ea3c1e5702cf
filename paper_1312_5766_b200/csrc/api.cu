// C ABI of libstrads_b200.so: argument checks, workspace carve-up and the order of kernels in a round.
// See include/strads.h for the contract of every entry point.
#include <climits>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "strads_internal.cuh"

using namespace strads;

// One scheduler thread of Section 3: its coefficients (Problem::part_index), its slice of the workspace
// (everything steps 1 and 2 write), and what orders its work against the updates.
struct Scheduler {
  alignas(64) unsigned char gram_tmap[128];   // tensor map over the BF16 copies of its candidates (dense layouts)
  Problem p;
  int walk_grid;             // CTAs of the cooperative on-demand walk (CSC)
  cudaStream_t stream;       // S > 1: steps 1 and 2 of its rounds are enqueued here
  cudaEvent_t block_ready;   // its block (the kept list) is complete
  cudaEvent_t updated;       // the update of its latest round is done: delta of its coefficients is final
};

struct strads_lasso_s {
  Scheduler sch[STRADS_MAX_SCHEDULERS];
  int n_sched;
  cudaStream_t stream;
  int device;
  long long round_host;     // the round index t (every round adds exactly one); scheduler t mod S is next
  // optional step timing: 6 events per round (start, after sample, pack, Gram, walk, update)
  cudaEvent_t* prof_events;
  long long prof_cap, prof_rounds;
  // strads_run replays captured launch sequences (fixed for a handle): eight rounds with one scheduler,
  // kGraphTurns turns of every scheduler, pipelined, with several
  cudaStream_t capture_stream;
  cudaGraph_t round_graph;
  cudaGraphExec_t round_exec;
  // one scheduler: shorter sequences (4, 2 and 1 rounds; with sampling ahead, from an early list) for what is left over
  cudaGraph_t tail_graph[3];
  cudaGraphExec_t tail_exec[3];
  cudaEvent_t fork;          // S > 1: where the schedulers' streams join the caller's stream
  // Sampling ahead (one scheduler; strads_run only): the draw of round t + 1 runs on its own stream beside the Gram
  // and walk of round t, and the round then starts from that list corrected for round t's update.
  bool ahead_ok;             // the configuration allows it
  Problem ahead;             // the early draw's view of the problem: own sampler state and buffers, P' + P winners
  cudaStream_t ahead_stream;
  cudaEvent_t ahead_fork, ahead_done;
  // ... and the whole-list retry of the dense Gram (launches that return at once unless the window was too short)
  // goes to a branch of its own, ending in its own gated copy of the update, instead of standing between the
  // window's walk and the update
  cudaStream_t retry_stream;
  cudaEvent_t retry_fork, retry_done;
  // ... and the correction of the next round's early list, beside the update
  cudaStream_t patch_stream;
  cudaEvent_t patch_fork, patch_done;
  // strads_round_host: beta and the residual travel on a stream of their own while the draw (which reads only the
  // priorities) already runs
  cudaStream_t copy_stream;
  cudaEvent_t copy_fork, copy_done;
  long long ahead_round;     // the round whose early list is in place (-1: none)
};

namespace {

constexpr int kProfEvents = 6;   // per round: start, after sample, pack, Gram, walk, update
constexpr int kGraphTurns = 16;  // S > 1: turns of every scheduler in the captured sequence
constexpr int kGraphRoundsAhead = 8;  // one scheduler, sampling ahead: rounds in the captured sequence
constexpr int kTailKinds = 3;         // and in the shorter ones for what is left over: 4, 2, 1 (a run of 20 rounds: 8 + 8 + 4)
constexpr int tail_rounds(int kind) { return kGraphRoundsAhead >> (kind + 1); }
static_assert(tail_rounds(kTailKinds - 1) == 1, "the shortest left-over sequence is one round");
static_assert(sizeof(strads_lasso_s::tail_exec) / sizeof(cudaGraphExec_t) == kTailKinds, "one slot per left-over sequence");
constexpr int kEdgeCap = 8192;        // conflicting pairs the Gram kernels can list for the walk (32 KB)
constexpr int kAheadMaxKeep = 4096;   // sampling ahead: the patch kernel holds 2 P keys in shared memory

Scheduler& on_turn(strads_lasso_s* h) { return h->sch[h->round_host % h->n_sched]; }

thread_local char g_cuda_err[256] = "";

int cuda_fail(cudaError_t e, const char* where) {
  snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", where, cudaGetErrorString(e));
  return STRADS_ERR_CUDA;
}
#define CK(call)                                            \
  do {                                                      \
    cudaError_t e__ = (call);                               \
    if (e__ != cudaSuccess) return cuda_fail(e__, #call);   \
  } while (0)

size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }
int pow2_ceil(int n) { int v = 1; while (v < n) v <<= 1; return v; }

struct Layout {
  size_t off_state, off_n2, off_hist, off_sure, off_boundary, off_cand, off_kept, off_kept_pos, off_dbeta, off_dbeta64,
      off_conflict, off_cand_dbeta64, off_cand_bnew, off_dot_partial, off_dot_ticket, off_margin, off_obj, off_amb, off_xcb, off_walk_blocked, off_walk_ctl, off_walk_cols,
      off_bucket_count, off_bucket_items, off_bucket_vals, off_bucket_cols, off_resid_acc, off_delta_prev, off_edges, off_patch_keys, off_cand_keys, off_survivors, off_bin_off, off_bin_cur, off_ahead_bin_off, off_ahead_bin_cur,
      off_ahead_state, off_ahead_hist, off_ahead_sure, off_ahead_boundary, off_ahead_keys, off_ahead_idx, total;
  int cap_sure, cap_boundary, mask_words, dot_parts, cap_amb, n_ahead, cap_ahead_boundary, cap_survivors;
  long long ldc, ldcb;
  bool buckets;
};

int n_sched_of(const strads_lasso_config_t* c) { return c->n_schedulers > 1 ? c->n_schedulers : 1; }

// Checks everything about cfg that does not need its pointers.
int check_sizes(const strads_lasso_config_t* c) {
  if (c == nullptr) return STRADS_ERR_INVALID_ARG;
  if (c->layout != STRADS_DENSE_COLMAJOR && c->layout != STRADS_CSC) return STRADS_ERR_BAD_LAYOUT;
  if (c->n_rows < 1 || c->n_cols < 1 || c->n_cols >= (1ll << 31) || c->n_rows >= (1ll << 31)) return STRADS_ERR_INVALID_ARG;
  if (c->layout == STRADS_DENSE_COLMAJOR && (c->ld < c->n_rows || (c->ld & 3) != 0)) return STRADS_ERR_BAD_LAYOUT;
  if (c->layout == STRADS_CSC && c->nnz < 0) return STRADS_ERR_INVALID_ARG;
  if (c->n_candidates < 1 || c->n_candidates > c->n_cols) return STRADS_ERR_INVALID_ARG;
  if (c->n_candidates > STRADS_MAX_CANDIDATES) return STRADS_ERR_UNSUPPORTED;
  if (c->n_keep < 1 || c->n_keep > c->n_candidates) return STRADS_ERR_INVALID_ARG;
  if (c->n_schedulers < 0 || c->n_schedulers > STRADS_MAX_SCHEDULERS) return STRADS_ERR_INVALID_ARG;
  if ((long long)c->n_candidates > c->n_cols / n_sched_of(c)) return STRADS_ERR_INVALID_ARG;   // smallest share: floor(J / S)
  return STRADS_OK;
}

// Slice of the workspace of one scheduler; the first one (`first`) also holds what all share
// (column norms, the objective's partial sums).
Layout carve(const strads_lasso_config_t* c, bool first = true) {
  Layout L;
  L.cap_sure = c->n_candidates;
  L.cap_boundary = pow2_ceil(c->n_candidates / 2 > 2048 ? c->n_candidates / 2 : 2048);
  L.mask_words = (c->n_candidates + 31) / 32;
  // CTAs per kept column in the dot kernel: about 1024 CTAs in all, so that every one of them is resident at
  // once (the kernel is a chain of dependent loads per CTA; residency, not depth per thread, hides it)
  long long parts = (1024 + c->n_keep - 1) / c->n_keep;
  const long long max_parts = c->n_rows / 2048 > 1 ? c->n_rows / 2048 : 1;
  if (parts > max_parts) parts = max_parts;
  L.dot_parts = (int)parts;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
  L.off_state = take(sizeof(DeviceState));
  L.off_n2 = take(first ? sizeof(double) * (size_t)c->n_cols : 0);
  L.off_hist = take(sizeof(unsigned int) * kHistBins);
  L.off_sure = take(sizeof(unsigned long long) * (size_t)L.cap_sure);
  L.off_boundary = take(sizeof(unsigned long long) * (size_t)L.cap_boundary);
  L.off_cand = take(sizeof(int) * (size_t)c->n_candidates);
  L.off_kept = take(sizeof(int) * (size_t)c->n_keep);
  L.off_kept_pos = take(sizeof(int) * (size_t)c->n_keep);
  L.off_dbeta = take(sizeof(float) * (size_t)c->n_keep);
  L.off_dbeta64 = take(sizeof(double) * (size_t)c->n_keep);
  L.off_conflict = take(sizeof(unsigned int) * (size_t)c->n_candidates * L.mask_words);
  const bool dense = c->layout == STRADS_DENSE_COLMAJOR;
  L.off_cand_dbeta64 = take(dense ? sizeof(double) * (size_t)c->n_candidates : 0);
  L.off_cand_bnew = take(dense ? sizeof(float) * (size_t)c->n_candidates : 0);
  L.off_dot_partial = take(sizeof(double) * (size_t)c->n_keep * L.dot_parts);
  L.off_dot_ticket = take(sizeof(unsigned int) * (size_t)c->n_keep);
  L.off_margin = take(first && (c->flags & STRADS_FLAG_LOGISTIC) ? sizeof(float) * (size_t)c->n_rows : 0);
  L.off_obj = take(first ? sizeof(double) * 2 * kObjBlocks : 0);
  L.cap_amb = c->layout == STRADS_DENSE_COLMAJOR ? (1 << 18) : 0;   // pairs the BF16 screen leaves to the exact recheck (1 MB)
  L.off_amb = take(sizeof(unsigned int) * (size_t)L.cap_amb);
  L.ldc = (c->n_rows + 3) / 4 * 4;
  L.ldcb = (c->n_rows + 7) / 8 * 8;
  L.off_xcb = take(c->layout == STRADS_DENSE_COLMAJOR ? sizeof(unsigned short) * (size_t)c->n_candidates * L.ldcb : 0);
  const bool csc = c->layout == STRADS_CSC;                            // on-demand walk (CSC)
  L.off_walk_blocked = take(csc ? sizeof(unsigned int) * (size_t)L.mask_words : 0);
  L.off_walk_ctl = take(csc ? sizeof(WalkControl) : 0);
  L.off_walk_cols = take(csc ? sizeof(WalkColumn) * (size_t)c->n_candidates : 0);
  // CSC Gram by row buckets: provided for while the buckets' candidate lists stay below 64 MB (N <= 2^20; their values take as much)
  L.buckets = csc && (size_t)c->n_rows * kBucketSlots * sizeof(int) <= ((size_t)64 << 20);
  L.off_bucket_count = take(L.buckets ? sizeof(unsigned int) * (size_t)c->n_rows : 0);
  L.off_bucket_items = take(L.buckets ? sizeof(int) * (size_t)c->n_rows * kBucketSlots : 0);
  L.off_bucket_vals = take(L.buckets ? sizeof(float) * (size_t)c->n_rows * kBucketSlots : 0);
  L.off_bucket_cols = take(L.buckets ? sizeof(BucketColumn) * (size_t)c->n_candidates : 0);
  L.off_resid_acc = take(csc ? sizeof(long long) * (size_t)c->n_rows : 0);
  L.off_delta_prev = take(sizeof(float) * (size_t)c->n_keep);
  L.off_edges = take(sizeof(unsigned int) * kEdgeCap);
  L.off_patch_keys = take(sizeof(unsigned long long) * 2 * (size_t)c->n_keep);
  L.off_cand_keys = take(dense ? sizeof(unsigned long long) * 2 * (size_t)c->n_candidates : 0);
  // keys the sampler's guided first pass saves for its collect pass (many coefficients only): 8 P' of them
  L.cap_survivors = c->n_cols >= (1 << 19) ? 8 * c->n_candidates : 0;
  L.off_survivors = take(sizeof(unsigned long long) * (size_t)L.cap_survivors);
  L.off_bin_off = take(sizeof(int) * (kHistBins + 1));
  L.off_bin_cur = take(sizeof(unsigned int) * kHistBins);
  // sampling ahead (one scheduler, P <= kAheadMaxKeep): a second set of sampler buffers for P' + P winners.
  // Dense layouts only: measured on the CSC workloads, a draw running beside the round's many-CTA, latency-bound
  // Gram kernels did not shorten it (c4: 102 -> 106 us per round, c5: 350 -> 384 us; again with the on-demand walk cut
  // to one CTA per SM so that the draw has registers to run in: c4 99 -> 103 us, c5 230 -> 281 us).
  const bool ahead = first && n_sched_of(c) == 1 && c->n_keep <= kAheadMaxKeep && c->layout == STRADS_DENSE_COLMAJOR;
  const long long n_ahead = (long long)c->n_candidates + c->n_keep < c->n_cols ? (long long)c->n_candidates + c->n_keep : c->n_cols;
  L.n_ahead = ahead ? (int)n_ahead : 0;
  L.cap_ahead_boundary = ahead ? pow2_ceil(L.n_ahead / 2 > 2048 ? L.n_ahead / 2 : 2048) : 0;
  L.off_ahead_state = take(ahead ? sizeof(DeviceState) : 0);
  L.off_ahead_hist = take(ahead ? sizeof(unsigned int) * kHistBins : 0);
  L.off_ahead_sure = take(sizeof(unsigned long long) * (size_t)L.n_ahead);
  L.off_ahead_boundary = take(sizeof(unsigned long long) * (size_t)L.cap_ahead_boundary);
  L.off_ahead_keys = take(sizeof(unsigned long long) * (size_t)L.n_ahead);
  L.off_ahead_idx = take(sizeof(int) * (size_t)L.n_ahead);
  L.off_ahead_bin_off = take(ahead ? sizeof(int) * (kHistBins + 1) : 0);
  L.off_ahead_bin_cur = take(ahead ? sizeof(unsigned int) * kHistBins : 0);
  L.total = o;
  return L;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Conflict bits of all candidate pairs.  Dense: tensor-core kernel unless the FP32 Gram itself is wanted
// (debug output) or the SIMT kernel is asked for.
// n_total: length of the whole list (n_cand < n_total: a window).  *walked: the Gram kernel's last CTA also settles the
// walk (dense tensor-core window), so that the walk kernel behind it only runs if that CTA leaves it the job.
cudaError_t launch_gram(const Scheduler& sc, cudaStream_t s, const int* cand, int n_cand, int n_total, float* gram_dbg,
                        bool only_if_short, cudaEvent_t after_pack = nullptr, bool* walked = nullptr) {
  const Problem& p = sc.p;
  const bool window = n_cand < n_total;
  if (walked != nullptr) *walked = false;
  if (after_pack != nullptr && (p.layout == STRADS_CSC || gram_dbg != nullptr || (p.flags & STRADS_FLAG_SIMT_GRAM))) {
    const cudaError_t e = cudaEventRecord(after_pack, s);          // these paths have no pack kernel
    if (e != cudaSuccess) return e;
    after_pack = nullptr;
  }
  if (p.layout == STRADS_CSC) return launch_gram_csc(p, cand, n_cand, gram_dbg, only_if_short, window, s);
  if (gram_dbg != nullptr || (p.flags & STRADS_FLAG_SIMT_GRAM)) return launch_gram_dense_simt(p, cand, n_cand, gram_dbg, s);
  return launch_gram_dense_tc(p, sc.gram_tmap, cand, n_cand, n_total, only_if_short, window, after_pack, s, walked);
}

// The greedy walk stops at P kept, so it normally looks at little more than the first P candidates: form the
// conflict bits of a leading window only (1.5 P + 128, rounded to the Gram tile) and walk that.  The result is
// final when P are kept inside the window; otherwise the filter raises window_short and the whole-list
// Gram + walk, enqueued behind it, runs (it is a no-op otherwise).  Same kept set either way.
int window_of(const Problem& p, int n_cand) {
  if (p.flags & (STRADS_FLAG_FULL_GRAM | STRADS_FLAG_SIMT_GRAM)) return n_cand;
  // dense: every window column is streamed and multiplied, so the window is cut closer (room for one candidate in five
  // to be rejected); CSC: the window's cost is in the pairs that share a row, and a short window costs a whole-list walk
  const long long slack = p.layout == STRADS_DENSE_COLMAJOR ? (p.n_keep / 4 > 64 ? p.n_keep / 4 : 64) : p.n_keep / 2 + 128;
  const long long w = ((long long)p.n_keep + slack + 127) / 128 * 128;
  return w * 2 <= n_cand ? (int)w : n_cand;          // a window only pays when it is well below the list
}

// Everything on `s`, one launch behind the other (strads_run with sampling ahead puts the retry on a branch of its
// own instead: round_sampling_ahead).
int gram_and_filter(const Scheduler& sc, cudaStream_t s, const int* cand, int n_cand, float* gram_dbg,
                    cudaEvent_t after_pack = nullptr, cudaEvent_t after_gram = nullptr) {
  const Problem& p = sc.p;
  if (p.flags & STRADS_FLAG_NO_FILTER) {
    if (after_pack) CK(cudaEventRecord(after_pack, s));
    if (after_gram) CK(cudaEventRecord(after_gram, s));
    CK(launch_filter(p, cand, n_cand, n_cand, false, p.kept, s));
    return STRADS_OK;
  }
  const int window = gram_dbg != nullptr ? n_cand : window_of(p, n_cand);
  bool walked = false;
  CK(launch_gram(sc, s, cand, window, n_cand, gram_dbg, false, after_pack, &walked));
  if (after_gram) CK(cudaEventRecord(after_gram, s));
  cudaStream_t rs = s;
  CK(launch_filter(p, cand, window, n_cand, false, p.kept, rs, walked));
  if (window < n_cand) {
    if (p.layout == STRADS_CSC) {
      // whole list, conflict rows formed only for the candidates the walk keeps
      CK(launch_walk_csc(p, cand, n_cand, window, sc.walk_grid, true, p.kept, s));
    } else {
      CK(launch_gram(sc, rs, cand, n_cand, n_cand, nullptr, true));
      CK(launch_filter(p, cand, n_cand, n_cand, true, p.kept, rs));
    }
  }
  return STRADS_OK;
}

// whether this round's pack kernel ran before the update (tensor-core Gram): with one scheduler it has then left the
// would-be changes of all candidates
bool update_after_pack(const Problem& p, bool gram_exported) {
  return p.layout == STRADS_DENSE_COLMAJOR && !(p.flags & (STRADS_FLAG_NO_FILTER | STRADS_FLAG_SIMT_GRAM)) && !gram_exported;
}

// One round, every step on the caller's stream, by the scheduler whose turn it is.
// before_gram: an event steps 2 and 3 have to wait for (state still on its way from the host; the draw needs only delta).
int one_round(strads_lasso_s* h, const strads_round_out_t* out, cudaEvent_t before_gram = nullptr) {
  h->ahead_round = -1;                                 // delta changes without a new early list
  const Scheduler& sc = on_turn(h);
  const Problem& p = sc.p;
  cudaEvent_t* ev = (h->prof_events != nullptr && h->prof_rounds < h->prof_cap) ? h->prof_events + kProfEvents * h->prof_rounds : nullptr;
  if (ev) CK(cudaEventRecord(ev[0], h->stream));
  CK(launch_sample(p, p.cand, h->stream));
  if (before_gram != nullptr) CK(cudaStreamWaitEvent(h->stream, before_gram, 0));
  if (ev) CK(cudaEventRecord(ev[1], h->stream));
  {
    const int rc = gram_and_filter(sc, h->stream, p.cand, p.n_cand, out ? out->gram : nullptr, ev ? ev[2] : nullptr,
                                   ev ? ev[3] : nullptr);
    if (rc) return rc;
  }
  if (ev) CK(cudaEventRecord(ev[4], h->stream));
  CK(launch_update(p, p.kept, 1, update_after_pack(p, out && out->gram), h->stream));
  if (ev) { CK(cudaEventRecord(ev[5], h->stream)); h->prof_rounds += 1; }
  h->round_host += 1;
  if (out != nullptr) {
    if (out->cand) CK(cudaMemcpyAsync(out->cand, p.cand, sizeof(int) * p.n_cand, cudaMemcpyDeviceToDevice, h->stream));
    if (out->kept || out->dbeta || out->counts) CK(launch_export(p, p.kept, out->kept, out->dbeta, out->counts, h->stream));
  }
  return STRADS_OK;
}

// What follows a window whose Gram kernel could not finish the job (its last CTA left the walk to the walk kernel,
// or fewer than P were kept inside the window): the walk kernel on the window if asked for, the whole-list Gram and
// walk if the window was short, then the gated copies of the correction of the early list and of the update.
int retry_sequence(strads_lasso_s* h, const Scheduler& sc, int window, bool early_patch, cudaStream_t rs) {
  const Problem& p = sc.p;
  CK(launch_filter(p, p.cand, window, p.n_cand, false, p.kept, rs, true));
  CK(launch_gram(sc, rs, p.cand, p.n_cand, p.n_cand, nullptr, true));
  CK(launch_filter(p, p.cand, p.n_cand, p.n_cand, true, p.kept, rs));
  if (early_patch) CK(launch_sample_patch(p, h->ahead, p.cand, rs, true, 2));
  CK(launch_update(p, p.kept, 1, true, rs, 2));
  return STRADS_OK;
}

// One round of strads_run with one scheduler, sampling ahead.  `main`: candidates, Gram (whose last CTA walks), update;
// `ahead_stream`: the early draw of the next round, which reads delta and so lies between this round's candidates
// and its update.
// Where the pack kernel forms the keys of every candidate (dense tensor-core rounds), the early list of round t + 1 is
// corrected as soon as round t's kept list stands, on `patch_stream` beside round t's update, and have_list says that
// the candidates of this round are already in place.  Otherwise the correction opens round t + 1 (it needs the keys
// the update leaves) and have_list says that the early list is there.
// The retry of a window that did not suffice is a branch of its own (`retry_stream`) that ends in its own copies of
// the correction and the update, gated on DeviceState::route like the copies on `main`, so that exactly one of each
// runs.  (Tried and dropped: the branch as the body of a CUDA-graph IF node whose condition the window Gram's last CTA
// sets -- c2 44.0 -> 42.4 us per round, c3 unchanged: evaluating the node costs about what the launches that return at
// once do.  Nor does it help to let those launches test the flags before the chain's wait: what orders them is the
// launching of their CTAs, 4,096 for the pack and 528 with nearly all of an SM's shared memory for each Gram kernel.
// Also tried and dropped: the pack step taken apart between captured rounds -- the BF16 copies of the next window
// behind the correction of its list, beside this round's update, and the proposals (which need the residual that
// update leaves) on a stream of their own beside the next Gram, so that the path would be correction -> copies -> Gram.
// Same results, but the columns are read twice and the kernels that overlap share one memory system: c3 68 -> 86 us
// per round, c2 39 -> 42 us.)
int round_sampling_ahead(strads_lasso_s* h, bool have_list, cudaStream_t main) {
  const Scheduler& sc = h->sch[0];
  const Problem& p = sc.p;
  const bool early_patch = update_after_pack(p, false) && p.proposals;     // (also: the gated update is the single-kernel one)
  if (!have_list) CK(launch_sample(p, p.cand, main));
  else if (!early_patch) CK(launch_sample_patch(p, h->ahead, p.cand, main));
  CK(cudaEventRecord(h->ahead_fork, main));
  CK(cudaStreamWaitEvent(h->ahead_stream, h->ahead_fork, 0));
  CK(launch_sample(h->ahead, h->ahead.cand, h->ahead_stream));
  CK(cudaEventRecord(h->ahead_done, h->ahead_stream));
  const int window = window_of(p, p.n_cand);
  if (!early_patch || window >= p.n_cand || (p.flags & STRADS_FLAG_GRAM_3XTF32)) {
    // no window, or a Gram that does not walk: everything in a row
    const int rc = gram_and_filter(sc, main, p.cand, p.n_cand, nullptr);
    if (rc) return rc;
    CK(cudaStreamWaitEvent(main, h->ahead_done, 0));
    if (early_patch) {
      CK(cudaEventRecord(h->patch_fork, main));
      CK(cudaStreamWaitEvent(h->patch_stream, h->patch_fork, 0));
      CK(launch_sample_patch(p, h->ahead, p.cand, h->patch_stream, true, 0));
      CK(cudaEventRecord(h->patch_done, h->patch_stream));
    }
    CK(launch_update(p, p.kept, 1, update_after_pack(p, false), main));
    if (early_patch) CK(cudaStreamWaitEvent(main, h->patch_done, 0));
    h->round_host += 1;
    h->ahead_round = h->round_host;
    return STRADS_OK;
  }
  bool walked = false;
  CK(launch_gram(sc, main, p.cand, window, p.n_cand, nullptr, false, nullptr, &walked));
  if (!walked) return STRADS_ERR_INVALID_ARG;            // (early_patch implies the tensor-core screen, whose last CTA walks)
  CK(cudaStreamWaitEvent(main, h->ahead_done, 0));         // the draw is over: delta may change, and the early list stands
  CK(cudaEventRecord(h->retry_fork, main));
  CK(cudaStreamWaitEvent(h->retry_stream, h->retry_fork, 0));
  {
    const int rc = retry_sequence(h, sc, window, early_patch, h->retry_stream);
    if (rc) return rc;
  }
  CK(cudaEventRecord(h->retry_done, h->retry_stream));
  CK(cudaEventRecord(h->patch_fork, main));
  CK(cudaStreamWaitEvent(h->patch_stream, h->patch_fork, 0));
  CK(launch_sample_patch(p, h->ahead, p.cand, h->patch_stream, true, 1));
  CK(cudaEventRecord(h->patch_done, h->patch_stream));
  CK(launch_update(p, p.kept, 1, true, main, 1));                            // runs if the window sufficed
  CK(cudaStreamWaitEvent(main, h->patch_done, 0));
  CK(cudaStreamWaitEvent(main, h->retry_done, 0));
  h->round_host += 1;
  h->ahead_round = h->round_host;
  return STRADS_OK;
}

// `count` rounds with S > 1 schedulers, pipelined ("Properties of STRADS": taking turns leaves every
// scheduler S-fold more time to prepare its block).  Steps 1 and 2 of a round go to its scheduler's own
// stream and need only that scheduler's previous update; the updates follow one another on `main` in round
// order, each waiting for its block.  Blocks of up to S - 1 later rounds are therefore prepared while an
// update runs, with the results of running the rounds one by one.  Everything enqueued here is ordered
// before whatever is enqueued on `main` afterwards: the last operation of every scheduler stream is a
// block that an update on `main` waits for.
int pipelined_rounds(strads_lasso_s* h, long long count, cudaStream_t main) {
  bool joined[STRADS_MAX_SCHEDULERS] = {};
  CK(cudaEventRecord(h->fork, main));
  for (long long i = 0; i < count; ++i) {
    const int s = (int)(h->round_host % h->n_sched);
    const Scheduler& sc = h->sch[s];
    const Problem& p = sc.p;
    CK(cudaStreamWaitEvent(sc.stream, joined[s] ? sc.updated : h->fork, 0));
    joined[s] = true;
    CK(launch_sample(p, p.cand, sc.stream));
    const int rc = gram_and_filter(sc, sc.stream, p.cand, p.n_cand, nullptr);
    if (rc) return rc;
    CK(cudaEventRecord(sc.block_ready, sc.stream));
    CK(cudaStreamWaitEvent(main, sc.block_ready, 0));
    CK(launch_update(p, p.kept, 1, update_after_pack(p, false), main));
    CK(cudaEventRecord(sc.updated, main));
    h->round_host += 1;
  }
  return STRADS_OK;
}

// Workspace pointers of scheduler `s` of `S` (slice at `ws`, laid out by L); X, y, beta, resid, delta, the
// column norms and the objective's partial sums are those of the first scheduler.
void fill_problem(Problem& p, const strads_lasso_config_t* c, const Layout& L, char* ws, int s, int S, const Problem* first) {
  p.layout = c->layout; p.N = c->n_rows; p.J = c->n_cols; p.ld = c->ld;
  p.xv = c->x_values; p.xrow = c->x_row_idx; p.xptr = reinterpret_cast<const long long*>(c->x_col_ptr);
  p.nnz = c->layout == STRADS_CSC ? c->nnz : 0;
  p.y = c->y; p.beta = c->beta; p.resid = c->resid; p.delta = c->delta;
  p.lambda = c->lambda; p.eta = c->eta; p.rho = c->rho; p.c_init = c->c_init;
  p.n_cand = c->n_candidates; p.n_keep = c->n_keep; p.seed = c->seed; p.flags = c->flags;
  p.st = reinterpret_cast<DeviceState*>(ws + L.off_state);
  p.n2 = first ? first->n2 : reinterpret_cast<double*>(ws + L.off_n2);
  p.hist = reinterpret_cast<unsigned int*>(ws + L.off_hist);
  p.sure = reinterpret_cast<unsigned long long*>(ws + L.off_sure);
  p.boundary = reinterpret_cast<unsigned long long*>(ws + L.off_boundary);
  p.cap_sure = L.cap_sure; p.cap_boundary = L.cap_boundary;
  p.cand = reinterpret_cast<int*>(ws + L.off_cand);
  p.kept = reinterpret_cast<int*>(ws + L.off_kept);
  p.kept_pos = reinterpret_cast<int*>(ws + L.off_kept_pos);
  p.dbeta = reinterpret_cast<float*>(ws + L.off_dbeta);
  p.dbeta64 = reinterpret_cast<double*>(ws + L.off_dbeta64);
  p.conflict = reinterpret_cast<unsigned int*>(ws + L.off_conflict);
  p.mask_words = L.mask_words;
  p.dot_partial = reinterpret_cast<double*>(ws + L.off_dot_partial);
  p.dot_ticket = reinterpret_cast<unsigned int*>(ws + L.off_dot_ticket);
  p.dot_parts = L.dot_parts;
  p.margin = first ? first->margin : ((c->flags & STRADS_FLAG_LOGISTIC) ? reinterpret_cast<float*>(ws + L.off_margin) : nullptr);
  p.obj_partial = first ? first->obj_partial : reinterpret_cast<double*>(ws + L.off_obj);
  p.amb_pairs = reinterpret_cast<unsigned int*>(ws + L.off_amb);
  p.cap_amb = L.cap_amb;
  p.ldc = L.ldc;
  p.xcb = reinterpret_cast<unsigned short*>(ws + L.off_xcb);
  p.ldcb = L.ldcb;
  p.cand_dbeta64 = reinterpret_cast<double*>(ws + L.off_cand_dbeta64);
  p.cand_bnew = reinterpret_cast<float*>(ws + L.off_cand_bnew);
  // with one scheduler a round's steps follow one another on one stream, so r at pack time is r at update time;
  // with several, blocks are prepared while earlier updates still change r
  p.proposals = (c->layout == STRADS_DENSE_COLMAJOR && S == 1) ? 1 : 0;
  p.cand_cur = nullptr;
  p.walk_blocked = reinterpret_cast<unsigned int*>(ws + L.off_walk_blocked);
  p.walk_ctl = reinterpret_cast<WalkControl*>(ws + L.off_walk_ctl);
  p.walk_cols = reinterpret_cast<WalkColumn*>(ws + L.off_walk_cols);
  p.resid_acc = reinterpret_cast<long long*>(ws + L.off_resid_acc);
  p.bucket_count = L.buckets ? reinterpret_cast<unsigned int*>(ws + L.off_bucket_count) : nullptr;
  p.bucket_items = L.buckets ? reinterpret_cast<int*>(ws + L.off_bucket_items) : nullptr;
  p.bucket_vals = L.buckets ? reinterpret_cast<float*>(ws + L.off_bucket_vals) : nullptr;
  p.bucket_cols = L.buckets ? reinterpret_cast<BucketColumn*>(ws + L.off_bucket_cols) : nullptr;
  p.part_count = S; p.part_index = s;
  p.sm_count = first ? first->sm_count : 0;
  p.round_ptr = &p.st->round; p.round_ahead = 0;
  p.keys_out = nullptr;
  p.delta_prev = reinterpret_cast<float*>(ws + L.off_delta_prev);
  p.bin_off = reinterpret_cast<int*>(ws + L.off_bin_off);
  p.bin_cur = reinterpret_cast<unsigned int*>(ws + L.off_bin_cur);
  p.survivors = L.cap_survivors ? reinterpret_cast<unsigned long long*>(ws + L.off_survivors) : nullptr;
  p.cap_survivors = L.cap_survivors;
  p.edges = reinterpret_cast<unsigned int*>(ws + L.off_edges);
  // (only the draw made ahead needs them: one scheduler, dense)
  p.patch_keys = (S == 1 && c->layout == STRADS_DENSE_COLMAJOR && c->n_keep <= kAheadMaxKeep)
                     ? reinterpret_cast<unsigned long long*>(ws + L.off_patch_keys) : nullptr;
  p.cand_keys = reinterpret_cast<unsigned long long*>(ws + L.off_cand_keys);
  p.cap_edges = kEdgeCap;
  p.wait_limit = 0; p.stall = 0;
}

// The early draw's view: everything of scheduler 0, except its own sampler state and buffers, P' + P winners with
// their keys, and the round index one ahead of the round in progress.
void fill_ahead(Problem& a, const Problem& p0, const Layout& L, char* ws) {
  a = p0;
  a.st = reinterpret_cast<DeviceState*>(ws + L.off_ahead_state);
  a.hist = reinterpret_cast<unsigned int*>(ws + L.off_ahead_hist);
  a.sure = reinterpret_cast<unsigned long long*>(ws + L.off_ahead_sure);
  a.boundary = reinterpret_cast<unsigned long long*>(ws + L.off_ahead_boundary);
  a.cap_sure = L.n_ahead; a.cap_boundary = L.cap_ahead_boundary;
  a.n_cand = L.n_ahead;
  a.cand = reinterpret_cast<int*>(ws + L.off_ahead_idx);
  a.keys_out = reinterpret_cast<unsigned long long*>(ws + L.off_ahead_keys);
  a.round_ptr = &p0.st->round; a.round_ahead = 1;
  a.bin_off = reinterpret_cast<int*>(ws + L.off_ahead_bin_off);
  a.bin_cur = reinterpret_cast<unsigned int*>(ws + L.off_ahead_bin_cur);
  a.survivors = nullptr; a.cap_survivors = 0;         // (the early draw is off the round's path: it keeps to the plain passes)
}

void release(strads_lasso_s* h) {
  for (int s = 0; s < STRADS_MAX_SCHEDULERS; ++s) {
    if (h->sch[s].stream != nullptr) cudaStreamDestroy(h->sch[s].stream);
    if (h->sch[s].block_ready != nullptr) cudaEventDestroy(h->sch[s].block_ready);
    if (h->sch[s].updated != nullptr) cudaEventDestroy(h->sch[s].updated);
  }
  if (h->fork != nullptr) cudaEventDestroy(h->fork);
  if (h->ahead_stream != nullptr) cudaStreamDestroy(h->ahead_stream);
  if (h->ahead_fork != nullptr) cudaEventDestroy(h->ahead_fork);
  if (h->ahead_done != nullptr) cudaEventDestroy(h->ahead_done);
  if (h->retry_stream != nullptr) cudaStreamDestroy(h->retry_stream);
  if (h->retry_fork != nullptr) cudaEventDestroy(h->retry_fork);
  if (h->retry_done != nullptr) cudaEventDestroy(h->retry_done);
  if (h->patch_stream != nullptr) cudaStreamDestroy(h->patch_stream);
  if (h->patch_fork != nullptr) cudaEventDestroy(h->patch_fork);
  if (h->patch_done != nullptr) cudaEventDestroy(h->patch_done);
  if (h->copy_stream != nullptr) cudaStreamDestroy(h->copy_stream);
  if (h->copy_fork != nullptr) cudaEventDestroy(h->copy_fork);
  if (h->copy_done != nullptr) cudaEventDestroy(h->copy_done);
  if (h->round_exec != nullptr) cudaGraphExecDestroy(h->round_exec);
  if (h->round_graph != nullptr) cudaGraphDestroy(h->round_graph);
  for (int k = 0; k < kTailKinds; ++k) {
    if (h->tail_exec[k] != nullptr) cudaGraphExecDestroy(h->tail_exec[k]);
    if (h->tail_graph[k] != nullptr) cudaGraphDestroy(h->tail_graph[k]);
  }
  if (h->capture_stream != nullptr) cudaStreamDestroy(h->capture_stream);
  delete h;
}

}  // namespace

extern "C" {

int strads_workspace_bytes(const strads_lasso_config_t* cfg, size_t* out_bytes) {
  if (out_bytes == nullptr) return STRADS_ERR_INVALID_ARG;
  const int rc = check_sizes(cfg);
  if (rc) return rc;
  *out_bytes = carve(cfg).total + (size_t)(n_sched_of(cfg) - 1) * carve(cfg, false).total;
  return STRADS_OK;
}

int strads_lasso_init(const strads_lasso_config_t* c, strads_handle_t* out_handle) {
  if (out_handle == nullptr) return STRADS_ERR_INVALID_ARG;
  *out_handle = nullptr;
  int rc = check_sizes(c);
  if (rc) return rc;
  if (!c->x_values || !c->y || !c->beta || !c->resid || !c->delta || !c->workspace) return STRADS_ERR_INVALID_ARG;
  if (c->layout == STRADS_CSC && (!c->x_row_idx || !c->x_col_ptr)) return STRADS_ERR_INVALID_ARG;
  if (!aligned(c->x_values, 16) || !aligned(c->y, 16) || !aligned(c->resid, 16) || !aligned(c->delta, 16) ||
      !aligned(c->beta, 4) || !aligned(c->workspace, 256))
    return STRADS_ERR_INVALID_ARG;
  if (!(c->lambda >= 0.f) || !(c->eta > 0.f) || !(c->rho > 0.f) || !(c->c_init > 0.f)) return STRADS_ERR_INVALID_ARG;
  if (!std::isfinite(c->lambda) || !std::isfinite(c->eta) || !std::isfinite(c->c_init)) return STRADS_ERR_INVALID_ARG;
  // the weight C^2 + eta must stay finite in binary32, or every never-updated coefficient's race time is 0 and the
  // first phase turns from a randomised sweep into one in index order
  if (c->c_init > STRADS_MAX_C_INIT) return STRADS_ERR_INVALID_ARG;
  const int S = n_sched_of(c);
  const Layout L = carve(c), Lrest = carve(c, false);
  if (c->workspace_bytes < L.total + (size_t)(S - 1) * Lrest.total) return STRADS_ERR_WORKSPACE_TOO_SMALL;

  strads_lasso_s* h = new (std::nothrow) strads_lasso_s();     // value-initialised: every pointer null
  if (h == nullptr) return STRADS_ERR_INVALID_ARG;
  h->n_sched = S;
  h->stream = static_cast<cudaStream_t>(c->stream);
  h->round_host = 0;
  auto fail = [&](int code) { release(h); return code; };
  cudaError_t e = cudaGetDevice(&h->device);
  if (e != cudaSuccess) return fail(cuda_fail(e, "cudaGetDevice"));
  int sm_count = 0;
  e = cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, h->device);
  if (e != cudaSuccess) return fail(cuda_fail(e, "cudaDeviceGetAttribute"));

  char* ws = static_cast<char*>(c->workspace);
  for (int s = 0; s < S; ++s) {
    Problem& p = h->sch[s].p;
    fill_problem(p, c, s == 0 ? L : Lrest, s == 0 ? ws : ws + L.total + (size_t)(s - 1) * Lrest.total, s, S,
                 s == 0 ? nullptr : &h->sch[0].p);
    p.sm_count = sm_count;
  }
  const Problem& p0 = h->sch[0].p;
  if ((e = prepare_sample(p0)) != cudaSuccess) return fail(cuda_fail(e, "prepare_sample"));
  if ((e = prepare_filter(p0)) != cudaSuccess) return fail(cuda_fail(e, "prepare_filter"));
  if ((e = prepare_gram_dense_tc()) != cudaSuccess) return fail(cuda_fail(e, "prepare_gram_dense_tc"));
  if ((e = launch_init(p0, h->stream)) != cudaSuccess) return fail(cuda_fail(e, "launch_init"));
  if ((e = launch_resid_from_beta(p0, h->stream)) != cudaSuccess) return fail(cuda_fail(e, "launch_resid_from_beta"));
  if ((e = cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking)) != cudaSuccess ||
      (e = cudaEventCreateWithFlags(&h->copy_fork, cudaEventDisableTiming)) != cudaSuccess ||
      (e = cudaEventCreateWithFlags(&h->copy_done, cudaEventDisableTiming)) != cudaSuccess)
    return fail(cuda_fail(e, "copy stream"));
  h->ahead_round = -1;
  h->ahead_ok = L.n_ahead > 0;
  if (h->ahead_ok) {
    fill_ahead(h->ahead, p0, L, ws);
    if ((e = launch_init_scheduler(h->ahead, p0, h->stream)) != cudaSuccess) return fail(cuda_fail(e, "launch_init_scheduler"));
    int prio_least = 0, prio_greatest = 0;             // the early draw yields to the round's own kernels
    if ((e = cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest)) != cudaSuccess) return fail(cuda_fail(e, "priority range"));
    if ((e = cudaStreamCreateWithPriority(&h->ahead_stream, cudaStreamNonBlocking, prio_least)) != cudaSuccess ||
        (e = cudaEventCreateWithFlags(&h->ahead_fork, cudaEventDisableTiming)) != cudaSuccess ||
        (e = cudaEventCreateWithFlags(&h->ahead_done, cudaEventDisableTiming)) != cudaSuccess ||
        (e = cudaStreamCreateWithPriority(&h->retry_stream, cudaStreamNonBlocking, prio_least)) != cudaSuccess ||
        (e = cudaEventCreateWithFlags(&h->retry_fork, cudaEventDisableTiming)) != cudaSuccess ||
        (e = cudaEventCreateWithFlags(&h->retry_done, cudaEventDisableTiming)) != cudaSuccess ||
        (e = cudaStreamCreateWithPriority(&h->patch_stream, cudaStreamNonBlocking, prio_greatest)) != cudaSuccess ||
        (e = cudaEventCreateWithFlags(&h->patch_fork, cudaEventDisableTiming)) != cudaSuccess ||
        (e = cudaEventCreateWithFlags(&h->patch_done, cudaEventDisableTiming)) != cudaSuccess)
      return fail(cuda_fail(e, "sampling-ahead stream"));
  }
  for (int s = 0; s < S; ++s) {
    Scheduler& sc = h->sch[s];
    if (sc.p.layout == STRADS_DENSE_COLMAJOR && (e = encode_gram_tensor_map(sc.p, sc.gram_tmap)) != cudaSuccess)
      return fail(cuda_fail(e, "encode_gram_tensor_map"));
    if (sc.p.layout == STRADS_CSC) {
      if ((e = prepare_walk_csc(sc.p, &sc.walk_grid)) != cudaSuccess) return fail(cuda_fail(e, "prepare_walk_csc"));
      if ((e = cudaMemsetAsync(sc.p.walk_ctl, 0, sizeof(WalkControl), h->stream)) != cudaSuccess)
        return fail(cuda_fail(e, "cudaMemsetAsync"));
      if ((e = cudaMemsetAsync(sc.p.resid_acc, 0, sizeof(long long) * (size_t)sc.p.N, h->stream)) != cudaSuccess)
        return fail(cuda_fail(e, "cudaMemsetAsync"));
      if (sc.p.bucket_count != nullptr &&
          (e = cudaMemsetAsync(sc.p.bucket_count, 0, sizeof(unsigned int) * (size_t)sc.p.N, h->stream)) != cudaSuccess)
        return fail(cuda_fail(e, "cudaMemsetAsync"));
    }
    if (s > 0 && (e = launch_init_scheduler(sc.p, p0, h->stream)) != cudaSuccess)
      return fail(cuda_fail(e, "launch_init_scheduler"));
    if (S > 1) {
      if ((e = cudaStreamCreateWithFlags(&sc.stream, cudaStreamNonBlocking)) != cudaSuccess ||
          (e = cudaEventCreateWithFlags(&sc.block_ready, cudaEventDisableTiming)) != cudaSuccess ||
          (e = cudaEventCreateWithFlags(&sc.updated, cudaEventDisableTiming)) != cudaSuccess)
        return fail(cuda_fail(e, "scheduler stream"));
    }
  }
  if (S > 1 && (e = cudaEventCreateWithFlags(&h->fork, cudaEventDisableTiming)) != cudaSuccess)
    return fail(cuda_fail(e, "cudaEventCreate"));
  *out_handle = h;
  return STRADS_OK;
}

int strads_round(strads_handle_t h, const strads_round_out_t* out) {
  if (h == nullptr) return STRADS_ERR_INVALID_ARG;
  return one_round(h, out);
}

// Rounds that one launch of the captured sequence runs.
static long long graph_rounds(const strads_lasso_s* h) {
  return h->n_sched > 1 ? (long long)kGraphTurns * h->n_sched : kGraphRoundsAhead;
}

// Captures the launch sequence of graph_rounds() rounds into a graph (on a private stream: the caller's may be
// the legacy default stream, which cannot be captured; nothing executes during capture).  With several
// schedulers the sequence starts with scheduler 0.  `tail_kind` >= 0: one of the shorter sequences from an early
// list instead (sampling ahead).
static int build_round_graph(strads_lasso_s* h, int tail_kind = -1) {
  const bool tail = tail_kind >= 0;
  if (h->capture_stream == nullptr) {
    int prio_least = 0, prio_greatest = 0;
    CK(cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest));
    CK(cudaStreamCreateWithPriority(&h->capture_stream, cudaStreamNonBlocking, prio_greatest));
  }
  cudaStream_t user = h->stream;
  const long long round_before = h->round_host;
  h->stream = h->capture_stream;
  cudaError_t e = cudaStreamBeginCapture(h->capture_stream, cudaStreamCaptureModeThreadLocal);
  int rc = STRADS_OK;
  if (e == cudaSuccess) {
    const long long ahead_before = h->ahead_round;
    if (h->n_sched > 1) {
      rc = pipelined_rounds(h, graph_rounds(h), h->capture_stream);
    } else if (h->ahead_ok) {
      const long long n = tail ? tail_rounds(tail_kind) : graph_rounds(h);
      for (long long i = 0; i < n && rc == STRADS_OK; ++i) rc = round_sampling_ahead(h, true, h->capture_stream);
    } else {
      const long long n = tail ? tail_rounds(tail_kind) : graph_rounds(h);
      for (long long i = 0; i < n && rc == STRADS_OK; ++i) rc = one_round(h, nullptr);
    }
    e = cudaStreamEndCapture(h->capture_stream, tail ? &h->tail_graph[tail_kind] : &h->round_graph);
    h->ahead_round = ahead_before;
  }
  h->stream = user;
  h->round_host = round_before;
  if (rc) return rc;
  if (e != cudaSuccess) return cuda_fail(e, "stream capture of a round");
  // instantiated and uploaded now, so that the first launch does not pay for either
  cudaGraphExec_t* exec = tail ? &h->tail_exec[tail_kind] : &h->round_exec;
  CK(cudaGraphInstantiate(exec, tail ? h->tail_graph[tail_kind] : h->round_graph, 0));
  CK(cudaGraphUpload(*exec, user));
  return STRADS_OK;
}

int strads_run(strads_handle_t h, int64_t n_rounds) {
  if (h == nullptr || n_rounds < 0) return STRADS_ERR_INVALID_ARG;
  if (h->n_sched > 1) {
    // whole captured sequences where they fit (they start with scheduler 0), the rest enqueued directly
    const long long R = graph_rounds(h);
    long long left = n_rounds;
    while (left > 0) {
      if (h->round_host % h->n_sched == 0 && left >= R) {
        if (h->round_exec == nullptr) {
          const int rc = build_round_graph(h);
          if (rc) return rc;
        }
        CK(cudaGraphLaunch(h->round_exec, h->stream));
        h->round_host += R;
        left -= R;
      } else {
        const long long to_turn0 = h->n_sched - h->round_host % h->n_sched;
        const long long count = left < R ? left : to_turn0;
        const int rc = pipelined_rounds(h, count, h->stream);
        if (rc) return rc;
        left -= count;
      }
    }
    return STRADS_OK;
  }
  const bool use_graph = h->prof_events == nullptr && n_rounds > 1;   // step timing needs events between kernels
  if (use_graph && h->round_exec == nullptr) {
    const int rc = build_round_graph(h);
    if (rc) return rc;
  }
  for (int k = 0; use_graph && k < kTailKinds; ++k) {
    if (h->tail_exec[k] != nullptr) continue;
    const int rc = build_round_graph(h, k);
    if (rc) return rc;
  }
  const long long R = graph_rounds(h);
  for (int64_t i = 0; i < n_rounds; ++i) {
    if (use_graph) {
      // (without sampling ahead every round draws its own list: nothing to have in place)
      const bool have_list = !h->ahead_ok || h->ahead_round == h->round_host;
      if (have_list && n_rounds - i >= R) {            // the early list of this round is in place: captured rounds
        CK(cudaGraphLaunch(h->round_exec, h->stream));
        h->round_host += R;
        h->ahead_round = h->round_host;
        i += R - 1;
      } else if (have_list) {                          // fewer rounds left than a sequence holds: the longest shorter one
        int k = 0;
        while (tail_rounds(k) > n_rounds - i) ++k;     // (the last kind is one round)
        CK(cudaGraphLaunch(h->tail_exec[k], h->stream));
        h->round_host += tail_rounds(k);
        h->ahead_round = h->round_host;
        i += tail_rounds(k) - 1;
      } else {                                         // first round of a run: draw now, start drawing ahead
        const int rc = round_sampling_ahead(h, false, h->stream);
        if (rc) return rc;
      }
    } else {
      const int rc = one_round(h, nullptr);
      if (rc) return rc;
    }
  }
  return STRADS_OK;
}

int strads_round_host(strads_handle_t h, float* beta_host, float* resid_host, float* delta_host,
                      int32_t* kept_host, float* dbeta_host, int32_t* counts_host) {
  if (h == nullptr || !beta_host || !resid_host || !delta_host) return STRADS_ERR_INVALID_ARG;
  const Problem& p = on_turn(h).p;
  if (p.flags & STRADS_FLAG_LOGISTIC) return STRADS_ERR_UNSUPPORTED;      // (the margin lives on the device)
  // delta first, on the handle's stream: the draw can start as soon as it is there; beta and the residual follow on
  // a second stream (behind whatever the handle's stream still has in flight) and are awaited before the Gram
  CK(cudaEventRecord(h->copy_fork, h->stream));
  CK(cudaStreamWaitEvent(h->copy_stream, h->copy_fork, 0));
  CK(cudaMemcpyAsync(p.delta, delta_host, sizeof(float) * p.J, cudaMemcpyHostToDevice, h->stream));
  CK(cudaMemcpyAsync(p.resid, resid_host, sizeof(float) * p.N, cudaMemcpyHostToDevice, h->copy_stream));
  CK(cudaMemcpyAsync(p.beta, beta_host, sizeof(float) * p.J, cudaMemcpyHostToDevice, h->copy_stream));
  CK(cudaEventRecord(h->copy_done, h->copy_stream));
  const int rc = one_round(h, nullptr, h->copy_done);
  if (rc) return rc;
  CK(cudaMemcpyAsync(beta_host, p.beta, sizeof(float) * p.J, cudaMemcpyDeviceToHost, h->stream));
  CK(cudaMemcpyAsync(resid_host, p.resid, sizeof(float) * p.N, cudaMemcpyDeviceToHost, h->stream));
  CK(cudaMemcpyAsync(delta_host, p.delta, sizeof(float) * p.J, cudaMemcpyDeviceToHost, h->stream));
  if (kept_host) CK(cudaMemcpyAsync(kept_host, p.kept, sizeof(int) * p.n_keep, cudaMemcpyDeviceToHost, h->stream));
  if (dbeta_host) CK(cudaMemcpyAsync(dbeta_host, p.dbeta, sizeof(float) * p.n_keep, cudaMemcpyDeviceToHost, h->stream));
  if (counts_host) CK(cudaMemcpyAsync(counts_host, p.st->counts, sizeof(int) * 4, cudaMemcpyDeviceToHost, h->stream));
  CK(cudaStreamSynchronize(h->stream));
  return STRADS_OK;
}

int strads_objective(strads_handle_t h, double* host_out) {
  if (h == nullptr || host_out == nullptr) return STRADS_ERR_INVALID_ARG;
  CK(launch_objective(h->sch[0].p, h->stream));
  CK(cudaMemcpyAsync(host_out, &h->sch[0].p.st->objective, sizeof(double), cudaMemcpyDeviceToHost, h->stream));
  CK(cudaStreamSynchronize(h->stream));
  return STRADS_OK;
}

int strads_sample(strads_handle_t h, int32_t* cand_dev) {
  if (h == nullptr || cand_dev == nullptr) return STRADS_ERR_INVALID_ARG;
  CK(launch_sample(on_turn(h).p, cand_dev, h->stream));
  return STRADS_OK;
}

int strads_filter(strads_handle_t h, const int32_t* cand_dev, int32_t n_cand, int32_t* kept_dev, int32_t* counts_dev,
                  float* gram_dev_or_null) {
  if (h == nullptr || cand_dev == nullptr || kept_dev == nullptr) return STRADS_ERR_INVALID_ARG;
  const Scheduler& sc = on_turn(h);
  if (n_cand < 0 || n_cand > sc.p.n_cand) return STRADS_ERR_INVALID_ARG;
  h->ahead_round = -1;                                 // (the early list is corrected from the last round's kept list)
  CK(launch_set_counts(sc.p, n_cand, 0, 0, h->stream));
  const int rc = gram_and_filter(sc, h->stream, cand_dev, n_cand, gram_dev_or_null);
  if (rc) return rc;
  CK(launch_export(sc.p, sc.p.kept, kept_dev, nullptr, counts_dev, h->stream));
  return STRADS_OK;
}

int strads_update(strads_handle_t h, const int32_t* kept_dev, int32_t n_kept, float* dbeta_dev) {
  if (h == nullptr) return STRADS_ERR_INVALID_ARG;
  const Problem& p = on_turn(h).p;
  if (n_kept < 0 || n_kept > p.n_keep || (n_kept > 0 && kept_dev == nullptr)) return STRADS_ERR_INVALID_ARG;
  h->ahead_round = -1;
  CK(launch_set_counts(p, n_kept, n_kept, n_kept, h->stream));
  if (n_kept > 0)
    CK(cudaMemcpyAsync(p.kept, kept_dev, sizeof(int) * n_kept, cudaMemcpyDeviceToDevice, h->stream));
  CK(launch_update(p, p.kept, 0, false, h->stream));
  if (dbeta_dev) CK(launch_export(p, p.kept, nullptr, dbeta_dev, nullptr, h->stream));
  return STRADS_OK;
}

int strads_get_round(strads_handle_t h, int64_t* t) {
  if (h == nullptr || t == nullptr) return STRADS_ERR_INVALID_ARG;
  *t = h->round_host;
  return STRADS_OK;
}

int strads_set_round(strads_handle_t h, int64_t t) {
  if (h == nullptr || t < 0) return STRADS_ERR_INVALID_ARG;
  h->round_host = t;
  h->ahead_round = -1;
  unsigned long long next[STRADS_MAX_SCHEDULERS];          // every scheduler's next turn at or after t
  for (int s = 0; s < h->n_sched; ++s) {
    next[s] = (unsigned long long)t + (unsigned long long)(((s - t % h->n_sched) + h->n_sched) % h->n_sched);
    CK(cudaMemcpyAsync(&h->sch[s].p.st->round, &next[s], sizeof(next[s]), cudaMemcpyHostToDevice, h->stream));
  }
  CK(cudaStreamSynchronize(h->stream));   // `next` lives on this stack frame
  return STRADS_OK;
}

int strads_totals(strads_handle_t h, int64_t* totals) {
  if (h == nullptr || totals == nullptr) return STRADS_ERR_INVALID_ARG;
  unsigned long long t[STRADS_MAX_SCHEDULERS][4];
  for (int s = 0; s < h->n_sched; ++s)
    CK(cudaMemcpyAsync(t[s], h->sch[s].p.st->totals, sizeof(t[s]), cudaMemcpyDeviceToHost, h->stream));
  CK(cudaStreamSynchronize(h->stream));
  for (int i = 0; i < 4; ++i) {
    totals[i] = 0;
    for (int s = 0; s < h->n_sched; ++s) totals[i] += (int64_t)t[s][i];
  }
  return STRADS_OK;
}

int strads_status(strads_handle_t h, uint32_t* bits_host_out) {
  if (h == nullptr) return STRADS_ERR_INVALID_ARG;
  unsigned int each[STRADS_MAX_SCHEDULERS] = {}, bits = 0;
  for (int s = 0; s < h->n_sched; ++s)
    CK(cudaMemcpyAsync(&each[s], &h->sch[s].p.st->status, sizeof(each[s]), cudaMemcpyDeviceToHost, h->stream));
  CK(cudaStreamSynchronize(h->stream));
  for (int s = 0; s < h->n_sched; ++s) bits |= each[s];
  if (bits_host_out) *bits_host_out = bits;
  if (bits & STRADS_STATUS_WAIT_EXPIRED) return STRADS_ERR_TIMEOUT;
  if (bits & STRADS_STATUS_NONFINITE) return STRADS_ERR_NUMERIC;
  return STRADS_OK;
}

// The captured launch sequence holds copies of the kernels' arguments: drop it when one of them changes.
static void drop_round_graph(strads_lasso_s* h) {
  if (h->round_exec != nullptr) { cudaGraphExecDestroy(h->round_exec); h->round_exec = nullptr; }
  if (h->round_graph != nullptr) { cudaGraphDestroy(h->round_graph); h->round_graph = nullptr; }
  for (int k = 0; k < kTailKinds; ++k) {
    if (h->tail_exec[k] != nullptr) { cudaGraphExecDestroy(h->tail_exec[k]); h->tail_exec[k] = nullptr; }
    if (h->tail_graph[k] != nullptr) { cudaGraphDestroy(h->tail_graph[k]); h->tail_graph[k] = nullptr; }
  }
}

int strads_set_wait_limit(strads_handle_t h, uint32_t iterations) {
  if (h == nullptr) return STRADS_ERR_INVALID_ARG;
  CK(cudaStreamSynchronize(h->stream));
  for (int s = 0; s < h->n_sched; ++s) h->sch[s].p.wait_limit = iterations;
  h->ahead.wait_limit = iterations;
  drop_round_graph(h);
  return STRADS_OK;
}

int strads_inject_stall(strads_handle_t h, int32_t which) {
  if (h == nullptr) return STRADS_ERR_INVALID_ARG;
  Scheduler& sc = on_turn(h);
  // only with a short limit in force: the stalled wait then gives up within milliseconds
  if (sc.p.wait_limit == 0 || sc.p.wait_limit > STRADS_STALL_MAX_WAIT_LIMIT) return STRADS_ERR_INVALID_ARG;
  if (which == STRADS_STALL_WALK_BARRIER) {
    if (sc.p.layout != STRADS_CSC) return STRADS_ERR_INVALID_ARG;
    // an arrival count no barrier of the walk can complete from
    CK(cudaMemsetAsync(&sc.p.walk_ctl->bar_count, 0x40, sizeof(unsigned int), h->stream));
  } else if (which == STRADS_STALL_GRAM_LOADS) {
    if (sc.p.layout != STRADS_DENSE_COLMAJOR) return STRADS_ERR_INVALID_ARG;
    sc.p.stall = 1;
    drop_round_graph(h);
  } else {
    return STRADS_ERR_INVALID_ARG;
  }
  return STRADS_OK;
}

int strads_recover(strads_handle_t h) {
  if (h == nullptr) return STRADS_ERR_INVALID_ARG;
  CK(cudaStreamSynchronize(h->stream));
  bool had_stall = false;
  for (int s = 0; s < h->n_sched; ++s) {
    Problem& p = h->sch[s].p;
    had_stall = had_stall || p.stall != 0;
    p.stall = 0;
    CK(cudaMemsetAsync(&p.st->status, 0, sizeof(unsigned int), h->stream));
    if (p.layout == STRADS_CSC) CK(cudaMemsetAsync(p.walk_ctl, 0, sizeof(WalkControl), h->stream));
  }
  if (had_stall) drop_round_graph(h);
  h->ahead_round = -1;                                   // (whatever was drawn ahead belongs to the abandoned rounds)
  CK(cudaStreamSynchronize(h->stream));
  return STRADS_OK;
}

int strads_margin(strads_handle_t h, float** dev_ptr_out) {
  if (h == nullptr || dev_ptr_out == nullptr || h->sch[0].p.margin == nullptr) return STRADS_ERR_INVALID_ARG;
  *dev_ptr_out = h->sch[0].p.margin;
  return STRADS_OK;
}

int strads_colnorm2(strads_handle_t h, const double** dev_ptr_out) {
  if (h == nullptr || dev_ptr_out == nullptr) return STRADS_ERR_INVALID_ARG;
  *dev_ptr_out = h->sch[0].p.n2;
  return STRADS_OK;
}

int strads_profile_begin(strads_handle_t h, int64_t max_rounds) {
  if (h == nullptr || max_rounds < 1 || max_rounds > (1 << 20)) return STRADS_ERR_INVALID_ARG;
  if (h->prof_events != nullptr || h->n_sched > 1) return STRADS_ERR_INVALID_ARG;
  h->prof_events = new (std::nothrow) cudaEvent_t[kProfEvents * max_rounds];
  if (h->prof_events == nullptr) return STRADS_ERR_INVALID_ARG;
  for (long long i = 0; i < kProfEvents * max_rounds; ++i) {
    cudaError_t e = cudaEventCreate(&h->prof_events[i]);
    if (e != cudaSuccess) {
      for (long long k = 0; k < i; ++k) cudaEventDestroy(h->prof_events[k]);
      delete[] h->prof_events;
      h->prof_events = nullptr;
      return cuda_fail(e, "cudaEventCreate");
    }
  }
  h->prof_cap = max_rounds;
  h->prof_rounds = 0;
  return STRADS_OK;
}

int strads_profile_end(strads_handle_t h, double* ms_host_out, int64_t* rounds_host_out) {
  if (h == nullptr || h->prof_events == nullptr) return STRADS_ERR_INVALID_ARG;
  int rc = STRADS_OK;
  cudaError_t e = cudaStreamSynchronize(h->stream);
  if (e != cudaSuccess) rc = cuda_fail(e, "cudaStreamSynchronize");
  double ms[kProfEvents - 1] = {0, 0, 0, 0, 0};
  for (long long r = 0; r < h->prof_rounds && rc == STRADS_OK; ++r)
    for (int k = 0; k < kProfEvents - 1; ++k) {
      float v = 0.f;
      e = cudaEventElapsedTime(&v, h->prof_events[kProfEvents * r + k], h->prof_events[kProfEvents * r + k + 1]);
      if (e != cudaSuccess) { rc = cuda_fail(e, "cudaEventElapsedTime"); break; }
      ms[k] += v;
    }
  if (ms_host_out) for (int k = 0; k < kProfEvents - 1; ++k) ms_host_out[k] = ms[k];
  if (rounds_host_out) *rounds_host_out = h->prof_rounds;
  for (long long i = 0; i < kProfEvents * h->prof_cap; ++i) cudaEventDestroy(h->prof_events[i]);
  delete[] h->prof_events;
  h->prof_events = nullptr; h->prof_cap = 0; h->prof_rounds = 0;
  return rc;
}

int strads_destroy(strads_handle_t h) {
  if (h == nullptr) return STRADS_ERR_INVALID_ARG;
  cudaStreamSynchronize(h->stream);
  if (h->prof_events != nullptr) {
    for (long long i = 0; i < kProfEvents * h->prof_cap; ++i) cudaEventDestroy(h->prof_events[i]);
    delete[] h->prof_events;
  }
  release(h);
  return STRADS_OK;
}

const char* strads_error_string(int code) {
  switch (code) {
    case STRADS_OK: return "ok";
    case STRADS_ERR_INVALID_ARG: return "invalid argument";
    case STRADS_ERR_BAD_LAYOUT: return "bad matrix layout";
    case STRADS_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case STRADS_ERR_CUDA: return "CUDA runtime error";
    case STRADS_ERR_NUMERIC: return "non-finite value met on the device";
    case STRADS_ERR_TIMEOUT: return "bounded device wait expired";
    case STRADS_ERR_UNSUPPORTED: return "size beyond a documented limit";
    default: return "unknown error";
  }
}

const char* strads_last_cuda_error(void) { return g_cuda_err; }

}  // extern "C"
