// Host side of the C ABI declared in include/dgs.h: argument checks, the layout of
// the caller's arena, and the kernel launches of one push / apply / pull event.
//
// Work runs on streams of the library's own so that independent steps of consecutive
// events overlap: pushes take kWorkerStreams worker streams in turn, the apply runs on a stream
// of its own, pulls take kServerStreams server streams in turn.  A push touches only the worker's
// velocity, the gradient and its own scratch; a pull touches one difference vector.  The
// small, latency-bound finalize kernels thus share the GPU with the bandwidth-bound passes
// of other events.  Order is kept by a small dependency tracker: every launch names the
// buffers it reads and writes, and waits (cudaStreamWaitEvent) for the last writer of what
// it reads and for the last writer and the readers of what it writes.  Per buffer the order
// of operations is therefore the order of the calls, which keeps the results bit-identical
// to a serial run.
#include "dgs.h"

#include <algorithm>
#include <cmath>
#include <cstddef>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "dgs_kernels.cuh"

using namespace dgs;

namespace {

constexpr uint64_t kAlign = 256;
constexpr uint32_t kMagic = 0x44475331u;  // "DGS1"
constexpr int kPushSlots = 8;  // push packet slots, used in turn (a slot is refilled once its apply has read it)
constexpr int kPullSlots = 6;             // pull packet slots
constexpr int kVarSlots = 4;              // packet slots of the pull without secondary compression
constexpr int kWorkerStreams = 4, kServerStreams = 6;   // library streams for the pushes and for the pulls
constexpr int kPushSets = kWorkerStreams;  // scratch sets and spare velocity buffers of the pushes
constexpr int kPullSets = kServerStreams;  // scratch sets of the pulls
constexpr int kAllSets = kPushSets + kPullSets;
constexpr int kLogRingMax = 128;            // most packets the apply log keeps
constexpr int kLogSlack = 32;               // slots of the log beyond one per worker
enum StreamId : int { kStW0 = 0, kStApply = kWorkerStreams, kStS0 = kWorkerStreams + 1,
                      kNumStreams = kWorkerStreams + 1 + kServerStreams };

inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

// Scratch of one selection pipeline ([0] push, on the worker stream; [1] pull, on the server stream)
struct ScratchLayout {
  uint64_t cand_idx, cand_val, part_cands, part_slot0, plan, part_live, cta_tot, seg_start;
  uint64_t hist1, hist2, hist3, sel, L_safe, L_wide, sync;
  uint64_t zero_begin, zero_end;  // [hist1, end of sync): cleared at init
};

struct Layout {
  uint64_t n_pad = 0;  // elements per state vector, padded to 256 bytes
  uint32_t num_tiles = 0;
  uint64_t K[2] = {0, 0};
  // byte offsets into the arena
  uint64_t theta, u, D, theta_local, grad_stage;
  uint64_t pkt_idx[kPushSlots + kPullSlots], pkt_val[kPushSlots + kPullSlots];  // push slots, then pull slots
  uint64_t var_idx[kVarSlots], var_val[kVarSlots], var_count[kVarSlots], L_one;
  uint64_t tiles, segs, seg_off, seg_tile0;
  ScratchLayout sc[kAllSets];  // push sets, then pull sets
  uint64_t L_next, u_slots, status, stats;
  uint64_t log_idx, log_val, log_bnd, log_pos;
  uint32_t log_ranges = 0;
  uint64_t blk_max;      // [N][blk_stride]: per block of kWarpTile elements, an upper bound on the keys of D_q in it
  uint64_t blk_stride = 0;  // ring of applied packets not yet folded into every D_q
  uint32_t log_ring = 0, log_stride = 0;
  uint64_t total = 0;
};

int check_config(const dgs_config* c) {
  if (!c || !c->segments) return DGS_EINVAL;
  if (c->n == 0 || c->n >= (1ull << 32)) return DGS_EINVAL;
  if (c->num_workers == 0 || c->num_workers > 65535) return DGS_EINVAL;
  if (c->num_segments == 0 || c->num_segments >= 65536) return DGS_EINVAL;
  if (c->pull_all_capacity > c->n) return DGS_EINVAL;
  if ((c->flags & DGS_PACKET_BF16) && (c->flags & DGS_PACKET_FP16)) return DGS_EINVAL;
  if (!std::isfinite(c->lr)) return DGS_EINVAL;
  if (!(c->momentum > 0.0f) || !(c->momentum <= 1.0f)) return DGS_EINVAL;
  uint64_t pos = 0;
  for (uint32_t s = 0; s < c->num_segments; ++s) {
    const dgs_segment& g = c->segments[s];
    if (g.offset != pos || g.len == 0) return DGS_EINVAL;
    if (g.k_push == 0 || g.k_push > g.len || g.k_pull == 0 || g.k_pull > g.len) return DGS_EINVAL;
    pos += g.len;
  }
  if (pos != c->n) return DGS_EINVAL;
  return DGS_OK;
}

// Tiles: every layer is cut at the global multiples of kWarpTile, so that all full
// tiles start 2 KB-aligned and only the first and last tile of a layer can be ragged.
void build_tiles(const dgs_config* c, std::vector<Tile>* tiles, std::vector<SegDesc>* segs) {
  uint32_t koff[2] = {0, 0};
  for (uint32_t s = 0; s < c->num_segments; ++s) {
    const dgs_segment& g = c->segments[s];
    SegDesc d;
    d.tile_begin = (uint32_t)tiles->size();
    uint64_t pos = g.offset, end = g.offset + g.len;
    uint32_t count = 0;
    while (pos < end) {
      const uint64_t next = std::min<uint64_t>(end, (pos / kWarpTile + 1) * kWarpTile);
      Tile t;
      t.start = (uint32_t)pos;
      t.len = (uint16_t)(next - pos);
      t.seg = (uint16_t)s;
      tiles->push_back(t);
      ++count;
      pos = next;
    }
    d.tile_end = d.tile_begin + count;
    d.k[0] = g.k_push;
    d.k[1] = g.k_pull;
    d.pkt_off[0] = koff[0];
    d.pkt_off[1] = koff[1];
    koff[0] += g.k_push;
    koff[1] += g.k_pull;
    segs->push_back(d);
  }
}

uint32_t count_tiles(const dgs_config* c) {
  uint64_t tiles = 0;
  for (uint32_t s = 0; s < c->num_segments; ++s) {
    const dgs_segment& g = c->segments[s];
    const uint64_t first = g.offset / kWarpTile, last = (g.offset + g.len - 1) / kWarpTile;
    tiles += last - first + 1;
  }
  return (uint32_t)tiles;
}

void make_layout(const dgs_config* c, Layout* L) {
  const uint64_t N = c->num_workers, S = c->num_segments;
  L->n_pad = align_up(c->n, kAlign / 4);
  L->num_tiles = count_tiles(c);
  L->K[0] = L->K[1] = 0;
  for (uint32_t s = 0; s < S; ++s) {
    L->K[0] += c->segments[s].k_push;
    L->K[1] += c->segments[s].k_pull;
  }
  uint64_t off = 0;
  auto take = [&](uint64_t bytes) {
    const uint64_t at = off;
    off = align_up(off + bytes, kAlign);
    return at;
  };
  const uint64_t vec = L->n_pad * 4;
  L->theta = take(vec);
  L->u = take(vec * (N + kPushSets));  // N velocities and the spares that pushes write into
  L->D = take(vec * N);
  L->theta_local = (c->flags & DGS_KEEP_LOCAL_MODEL) ? take(vec * N) : 0;
  L->grad_stage = (c->flags & DGS_HOST_IO) ? take(vec) : 0;
  for (int p = 0; p < kPushSlots + kPullSlots; ++p) {
    const uint64_t K = L->K[p < kPushSlots ? 0 : 1];
    L->pkt_idx[p] = take(K * 4);
    L->pkt_val[p] = take(K * 4);
  }
  for (int p = 0; p < kVarSlots; ++p) {
    L->var_idx[p] = c->pull_all_capacity ? take((uint64_t)c->pull_all_capacity * 4) : 0;
    L->var_val[p] = c->pull_all_capacity ? take((uint64_t)c->pull_all_capacity * 4) : 0;
    L->var_count[p] = c->pull_all_capacity ? take(4) : 0;
  }
  L->L_one = take(S * 4);
  L->tiles = take((uint64_t)L->num_tiles * sizeof(Tile));
  L->segs = take(S * sizeof(SegDesc));
  L->seg_off = take((S + 1) * 4);
  L->seg_tile0 = take(S * 4);
  for (int k = 0; k < kAllSets; ++k) {
    ScratchLayout& sc = L->sc[k];
    sc.cand_idx = take(vec);
    sc.cand_val = take(vec);
    sc.part_cands = take((uint64_t)kMaxGrid * 4);
    sc.part_slot0 = take((uint64_t)kMaxGrid * 4);
    sc.plan = take((uint64_t)(kMaxGrid + 1) * 4);
    sc.part_live = take((uint64_t)kMaxGrid * 4);
    sc.cta_tot = take((uint64_t)kMaxWorkers * sizeof(uint2));
    sc.seg_start = take(S * sizeof(uint2));
    sc.hist1 = take(S * kBins1 * 4);
    sc.zero_begin = sc.hist1;
    sc.hist2 = take(S * kBins2 * 4);
    sc.hist3 = take(S * kBins3 * 4);
    sc.sel = take(S * sizeof(SegSel));
    sc.L_safe = take(S * 4);
    sc.L_wide = take(S * 4);
    sc.sync = take(kNumSyncWords * 4);
    sc.zero_end = off;
  }
  // A slot of the log is reused `ring` packets later, and the apply that refills it waits for every catch-up that
  // still reads the old packet.  A worker that comes back after N events reads the N newest packets, so ring - N
  // is how many events the server side of an event may lag behind the pushes before the pushes stall.
  // (with irregular arrivals a worker is often away for more than N events -- one gap in eight is longer than 2 N when
  // every event's worker is drawn at random -- and a worker about to fall off the ring is caught up on the apply
  // stream, in the way of every later event: four rounds of room where that many packets fit the cap)
  L->log_ring = (uint32_t)std::min<uint64_t>(kLogRingMax, std::max<uint64_t>(std::max<uint64_t>(N + kLogSlack, 4 * N), 16));
  L->log_stride = (uint32_t)align_up(L->K[0], 64);
  L->log_idx = take((uint64_t)L->log_ring * L->log_stride * 4);
  L->log_val = take((uint64_t)L->log_ring * L->log_stride * 4);
  {
    // ranges of the log = CTAs of a catch-up: about kCatchTarget entries each when a worker has missed
    // as many packets as there are workers, and no more ranges than a packet has entries
    const uint64_t entries = std::min<uint64_t>(N, L->log_ring) * L->K[0];
    L->log_ranges = (uint32_t)std::min<uint64_t>(std::min<uint64_t>(kCatchMaxGrid, L->K[0]),
                                                 std::max<uint64_t>(1, (entries + kCatchTarget - 1) / kCatchTarget));
  }
  L->log_bnd = take((uint64_t)L->log_ranges * 4 * 2);   // two generations of ranges, see apply_impl
  L->log_pos = take((uint64_t)L->log_ring * (L->log_ranges + 1) * 4);
  L->blk_stride = align_up((c->n + kWarpTile - 1) / kWarpTile, 64);
  L->blk_max = take(N * L->blk_stride * 4);
  L->L_next = take(2 * N * S * 4);
  L->u_slots = take((N + kPushSets) * sizeof(float*));
  L->status = take(4);
  L->stats = take((uint64_t)kNumStats * 8);
  L->total = off;
}

}  // namespace

struct dgs_ctx {
  uint32_t magic;
  dgs_config cfg;
  std::vector<dgs_segment> segments;
  Layout lay;
  char* base;
  cudaStream_t user;       // the caller's stream: entry point of dependencies, target of dgs_flush
  cudaStream_t st[kNumStreams];
  cudaEvent_t ev_in;       // "everything the caller had enqueued when the call was made"
  bool forked[kNumStreams];  // stream already waits for ev_in of the current call
  cudaEvent_t ev_tail[kNumStreams];  // for dgs_flush
  // dependency tracker
  struct Dep {
    cudaEvent_t ev = nullptr;
    int stream = -1;
    uint64_t seq = 0;  // position of the task in the order of all tasks (0: none)
  };
  struct Res {
    Dep last_write;
    std::vector<Dep> reads;  // readers since the last write
  };
  std::vector<Res> res;
  // one "done" event per task, reused in turn; a ring per stream, so that an event is only ever
  // re-recorded later on the same stream and waiting for a reused one still covers the older task
  std::vector<cudaEvent_t> ev_ring[kNumStreams];
  size_t ev_next[kNumStreams];
  uint64_t task_seq;                               // tasks filed so far
  uint64_t waited_seq[kNumStreams][kNumStreams];   // [waiting stream][stream]: newest task already waited for
  uint64_t push_count, pull_count, event_count, var_count;
  // Lazy difference vectors: packet number p (counted from 0) of the library's own pushes sits in slot
  // p % ring of the log from its apply on; applied[q] packets have been folded into D_q so far.
  PacketLog log;
  uint64_t log_head;              // packets filed so far
  uint64_t last_ranges;           // packet number at which the current generation of ranges was taken
  int cur_gen;                    // generation of ranges that new packets are filed under
  int64_t gen_last[2];            // newest packet filed under each generation, -1 if none
  std::vector<uint8_t> slot_gen;  // per slot of the ring: generation its packet was filed under
  std::vector<uint64_t> applied;  // per worker
  Workspace ws[kAllSets];  // push sets, then pull sets
  float inv_m;
  int sms;               // SMs of the device
  // Which form of the pull's stream pass to launch.  The ring-less form wins when a pull reads a small part
  // of D_w (it holds almost no shared memory beside the push passes), the staged form when it reads most of
  // it.  The kernels count the chunks they cover and read; after every pull those two counters are copied
  // to pinned host memory on the pull's stream, and the host looks at whatever has arrived so far (never
  // waiting): a stale figure only means a less suitable form, the results are the same either way.
  bool multi_worker;
  unsigned long long* h_chunks;      // pinned: [0] chunks covered, [1] chunks read, as of some recent pull
  unsigned long long seen_chunks[2]; // the figures at the last decision
  bool light_now;
  int stream_grid[3];    // CTAs of the stand-alone stream pass, per mode
  int hist_grid[3];      // CTAs of the whole-input histogram pass, per mode
  int finalize_grid[3];  // CTAs of the cooperative finalize kernel, per mode
  int finalize_max[3];   // most CTAs of it that can be resident at once
  uint32_t select_seq;   // selections launched so far
  uint64_t kind_seq[2];  // selections of each kind launched so far
  // Carried bounds: row (kind, worker) of L_next holds the bounds suggested by that worker's
  // latest selection of that kind ([0] push, [1] pull).  row_age says in which state it was
  // made: pushes the worker had done before (push), packets accumulated in D_w since its
  // previous pull (pull).  Thresholds grow with that age, so a row made at an age no larger
  // than the current one is a safe-side guess; the most recent such row is used.
  std::vector<uint8_t> row_valid[2];
  std::vector<uint64_t> row_time[2], row_age[2];
  std::vector<uint64_t> pushes;  // pushes done per worker
  std::vector<int64_t> prev;
  uint64_t timestamp;
  uint64_t launches;
  int last_cuda;
  bool broken;
  // optional per-kernel timing (CUDA events on the launching stream)
  bool timing;
  std::vector<cudaEvent_t> ev_pool;   // pairs: [2i] start, [2i+1] stop
  std::vector<int> ev_kernel;         // kernel id of each recorded pair
  std::vector<int> ev_stream;         // index of the library stream it ran on
  double time_ms[DGS_NUM_KERNELS];
  uint64_t time_count[DGS_NUM_KERNELS];

  template <typename T>
  T* at(uint64_t off) const { return reinterpret_cast<T*>(base + off); }
  float* u_buf(uint32_t q) const { return at<float>(lay.u) + (uint64_t)q * lay.n_pad; }
  float* D_buf(uint32_t q) const { return at<float>(lay.D) + (uint64_t)q * lay.n_pad; }
  float* theta_local_buf(uint32_t q) const { return at<float>(lay.theta_local) + (uint64_t)q * lay.n_pad; }
  uint32_t* blk_max(uint32_t q) const { return at<uint32_t>(lay.blk_max) + (uint64_t)q * lay.blk_stride; }
  float** u_slot(uint32_t q) const { return at<float*>(lay.u_slots) + q; }
  uint32_t* L_next(int pm, uint32_t w) const {
    return at<uint32_t>(lay.L_next) + ((uint64_t)pm * cfg.num_workers + w) * cfg.num_segments;
  }
};

namespace {

// resources of the dependency tracker
struct ResIds {
  uint32_t N;
  uint32_t U(uint32_t w) const { return w; }
  uint32_t D(uint32_t q) const { return N + q; }
  uint32_t TL(uint32_t q) const { return 2 * N + q; }
  uint32_t ROW(int kind, uint32_t w) const { return 3 * N + (uint32_t)kind * N + w; }
  uint32_t THETA() const { return 5 * N; }
  uint32_t SPARE(int j) const { return 5 * N + 1 + j; }
  uint32_t SCR(int kind, int set) const { return 5 * N + 1 + kPushSets + (kind ? kPushSets : 0) + set; }
  uint32_t PKT(int slot) const { return 5 * N + 1 + kPushSets + kAllSets + slot; }   // push slots, then pull slots
  uint32_t VPKT(int slot) const { return PKT(kPushSlots + kPullSlots) + (uint32_t)slot; }
  uint32_t STAGE() const { return VPKT(kVarSlots); }
  uint32_t LOG(uint32_t slot) const { return STAGE() + 1 + slot; }
  uint32_t RANGES(int gen) const { return LOG(kLogRingMax) + (uint32_t)gen; }   // the two generations of ranges of the log
  uint32_t count() const { return RANGES(1) + 1; }
};

#define DGS_CUDA(ctx, call)                 \
  do {                                      \
    cudaError_t e_ = (call);                \
    if (e_ != cudaSuccess) {                \
      (ctx)->last_cuda = (int)e_;           \
      (ctx)->broken = true;                 \
      return DGS_ECUDA;                     \
    }                                       \
  } while (0)

inline int live(dgs_ctx* c) {
  if (!c || c->magic != kMagic) return DGS_ESTATE;
  if (c->broken) return DGS_ESTATE;
  return DGS_OK;
}

constexpr size_t kMaxTimedLaunches = 1 << 16;
constexpr int kFinalizeWorkers = 64;  // CTAs of the finalize kernel (more of them take SM slots from the stream passes)

// Records an event before and after one launch when timing is on.
struct TimedLaunch {
  dgs_ctx* c;
  cudaStream_t st;
  cudaEvent_t stop = nullptr;
  TimedLaunch(dgs_ctx* ctx, cudaStream_t stream, int kernel_id) : c(ctx), st(stream) {
    if (!c->timing || c->ev_kernel.size() >= kMaxTimedLaunches) return;
    const size_t i = c->ev_kernel.size();
    while (c->ev_pool.size() < 2 * (i + 1)) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return;
      c->ev_pool.push_back(e);
    }
    if (cudaEventRecord(c->ev_pool[2 * i], st) != cudaSuccess) return;
    stop = c->ev_pool[2 * i + 1];
    c->ev_kernel.push_back(kernel_id);
    int which = -1;
    for (int j = 0; j < kNumStreams; ++j)
      if (c->st[j] == st) which = j;
    c->ev_stream.push_back(which);
  }
  ~TimedLaunch() {
    if (stop) cudaEventRecord(stop, st);
  }
};

// Makes an internal stream wait for everything the caller had enqueued on its stream when the
// current API call began (ev_in is recorded once per call by begin_call).
int begin_call(dgs_ctx* c) {
  DGS_CUDA(c, cudaEventRecord(c->ev_in, c->user));
  for (int i = 0; i < kNumStreams; ++i) c->forked[i] = false;
  return DGS_OK;
}
int fork_from_user(dgs_ctx* c, int which) {
  if (c->forked[which]) return DGS_OK;
  DGS_CUDA(c, cudaStreamWaitEvent(c->st[which], c->ev_in, 0));
  c->forked[which] = true;
  return DGS_OK;
}

// Waits (on the host) for all internal streams and the caller's stream.
int sync_all(dgs_ctx* c) {
  for (int i = 0; i < kNumStreams; ++i) DGS_CUDA(c, cudaStreamSynchronize(c->st[i]));
  DGS_CUDA(c, cudaStreamSynchronize(c->user));
  return DGS_OK;
}

// A task = the launches of one step on one stream.  task_begin makes the stream wait for
// whatever the task depends on; task_end records the task's completion and files it with
// the buffers it touched.
struct Task {
  int stream;
  std::vector<uint32_t> reads, writes;
};
int task_begin(dgs_ctx* c, const Task& t) {
  // Tasks of one stream complete in order, so per stream only the newest task that this one depends
  // on matters, and only if the stream has not already waited for that task or a newer one.
  dgs_ctx::Dep need[kNumStreams];
  auto want = [&](const dgs_ctx::Dep& d) {
    if (!d.ev || d.stream == t.stream) return;   // same stream: already ordered
    if (d.seq > need[d.stream].seq) need[d.stream] = d;
  };
  for (uint32_t r : t.reads) want(c->res[r].last_write);
  for (uint32_t w : t.writes) {
    const dgs_ctx::Res& x = c->res[w];
    want(x.last_write);
    for (const dgs_ctx::Dep& rd : x.reads) want(rd);
  }
  for (int s = 0; s < kNumStreams; ++s) {
    if (!need[s].ev || need[s].seq <= c->waited_seq[t.stream][s]) continue;
    DGS_CUDA(c, cudaStreamWaitEvent(c->st[t.stream], need[s].ev, 0));
    c->waited_seq[t.stream][s] = need[s].seq;
  }
  return DGS_OK;
}
int task_end(dgs_ctx* c, const Task& t) {
  dgs_ctx::Dep d;
  d.ev = c->ev_ring[t.stream][c->ev_next[t.stream]];
  d.stream = t.stream;
  d.seq = ++c->task_seq;
  c->ev_next[t.stream] = (c->ev_next[t.stream] + 1) % c->ev_ring[t.stream].size();
  DGS_CUDA(c, cudaEventRecord(d.ev, c->st[t.stream]));
  for (uint32_t r : t.reads) c->res[r].reads.push_back(d);
  for (uint32_t w : t.writes) {
    dgs_ctx::Res& x = c->res[w];
    x.last_write = d;
    x.reads.clear();
  }
  return DGS_OK;
}

// Dependencies of folding the filed packets that D_q has not seen yet into it.
void catch_up_deps(const dgs_ctx* c, uint32_t q, Task* t) {
  const ResIds R{c->cfg.num_workers};
  bool gen_used[2] = {false, false};
  for (uint64_t p = c->applied[q]; p < c->log_head; ++p) {
    t->reads.push_back(R.LOG((uint32_t)(p % c->log.ring)));
    gen_used[c->slot_gen[p % c->log.ring]] = true;
  }
  for (int g = 0; g < 2; ++g)
    if (gen_used[g]) t->reads.push_back(R.RANGES(g));
  t->writes.push_back(R.D(q));
}
// The launch itself, on a stream that task_begin has prepared with those dependencies.
int catch_up_launch(dgs_ctx* c, uint32_t q, cudaStream_t st) {
  uint64_t first = c->applied[q];
  // The packets still to be folded in were filed under at most two generations of ranges, the older
  // ones first: one launch per generation and per kCatchMaxPackets packets, in that order (the order of
  // the subtractions is kept).
  while (first < c->log_head) {
    const int gen = c->slot_gen[first % c->log.ring];
    uint64_t end = first + 1;
    while (end < c->log_head && end - first < (uint64_t)kCatchMaxPackets && c->slot_gen[end % c->log.ring] == gen) ++end;
    const uint32_t count = (uint32_t)(end - first);
    TimedLaunch tl(c, st, DGS_KERNEL_CATCH_UP);
    // One CTA per SM at most, each taking several ranges in turn: the kernel runs beside the push passes of
    // later events, and the loop is faster when it holds few SM resources than when it finishes early.
    const unsigned catch_grid = std::min<unsigned>(c->log.ranges, (unsigned)c->sms);
    PacketLog lg = c->log;
    lg.bnd = c->log.bnd + (size_t)gen * c->log.ranges;
    k_catch_up<<<catch_grid, kCatchThreads, 0, st>>>(lg, first, count, c->D_buf(q), c->blk_max(q), c->cfg.n);
    DGS_CUDA(c, cudaGetLastError());
    c->launches += 1;
    first = end;
  }
  c->applied[q] = c->log_head;
  return DGS_OK;
}
// Both, as a task of its own on the apply stream.
int catch_up_now(dgs_ctx* c, uint32_t q) {
  if (c->applied[q] == c->log_head) return DGS_OK;
  Task t;
  t.stream = kStApply;
  catch_up_deps(c, q, &t);
  int rc = task_begin(c, t);
  if (rc != DGS_OK) return rc;
  rc = catch_up_launch(c, q, c->st[kStApply]);
  if (rc != DGS_OK) return rc;
  return task_end(c, t);
}

// Row of carried bounds for a selection of this kind at this age: the most recent row made at
// an age <= `age`, but preferably not one written by the selections that the other streams of
// this kind are still working on (waiting for those would chain the streams together; the row
// before them was written on this selection's own stream).  -1 if there is none.
int pick_row(const dgs_ctx* c, int kind, uint64_t age) {
  int best = -1, best_old = -1;
  const uint64_t in_flight = (uint64_t)(kind ? kServerStreams : kWorkerStreams) - 1;
  const uint64_t newest = c->kind_seq[kind];
  for (uint32_t q = 0; q < c->cfg.num_workers; ++q) {
    if (!c->row_valid[kind][q] || c->row_age[kind][q] > age) continue;
    const uint64_t t = c->row_time[kind][q];
    if (best < 0 || t < c->row_time[kind][best]) best = (int)q;   // else the oldest: the likeliest to be complete
    if (t + in_flight <= newest && (best_old < 0 || t > c->row_time[kind][best_old])) best_old = (int)q;
  }
  return best_old >= 0 ? best_old : best;
}

inline int packet_format_of(const dgs_ctx* c) {
  return (c->cfg.flags & DGS_PACKET_BF16) ? 1 : (c->cfg.flags & DGS_PACKET_FP16) ? 2 : 0;
}

// The form of the next pull's stream pass (see dgs_ctx::h_chunks): ring-less if the pulls counted since the
// last decision read less than a third of the chunks they covered.
bool use_light_pull(dgs_ctx* c) {
  if (!c->multi_worker || !c->h_chunks) return false;
  const unsigned long long covered = *(volatile unsigned long long*)&c->h_chunks[0];
  const unsigned long long read = *(volatile unsigned long long*)&c->h_chunks[1];
  if (covered > c->seen_chunks[0] && read >= c->seen_chunks[1]) {
    c->light_now = 3 * (read - c->seen_chunks[1]) < covered - c->seen_chunks[0];
    c->seen_chunks[0] = covered;
    c->seen_chunks[1] = read;
  }
  return c->light_now;
}
// After a pull: its counters on their way to the host (on the pull's stream, nobody waits for them).
int report_chunks(dgs_ctx* c, cudaStream_t st) {
  if (c->h_chunks)
    DGS_CUDA(c, cudaMemcpyAsync(c->h_chunks, c->ws[0].stats + 3, 2 * sizeof(unsigned long long), cudaMemcpyDeviceToHost, st));
  return DGS_OK;
}

template <int MODE>
int launch_select(dgs_ctx* c, const SelArgs& a_in, uint32_t worker, uint64_t age, int stream_id, int set,
                  Task& task) {
  constexpr int KIND = MODE == kPull ? 1 : 0;
  const ResIds R{c->cfg.num_workers};
  cudaStream_t st = c->st[stream_id];
  Workspace& ws = c->ws[(KIND ? kPushSets : 0) + set];
  SelArgs a = a_in;
  a.speculate = (c->cfg.flags & DGS_NO_SPECULATION) ? 0 : 1;
  int row = a.speculate ? pick_row(c, KIND, age) : -1;
  // A worker that comes straight back (no other worker's packet since its last pull) selects from what that pull
  // left plus its own packet, and no other pull's bound says anything about that: 44 % of such guesses admitted
  // fewer than k candidates (four workers drawn at random), each then starting over inside finalize.  The
  // histogram route costs less than that on average.  (With one worker every pull is like the one before it.)
  if (KIND == 1 && age < 2 && c->cfg.num_workers > 1) row = -1;
  const bool single_pass = row >= 0;
  a.L_next = c->L_next(KIND, worker);
  a.force_two_pass = single_pass ? 0 : 1;
  // A selection of very many entries (dense packets) gets more CTAs: one more per 4096 entries.  One whose
  // candidates (about three times the entries) fit the registers of 48 CTAs' threads, eight each, gets only
  // those 48: finalize runs beside the push passes of later events and should hold few SMs.
  int fin_base = c->finalize_grid[MODE];
  if (3ull * a.pkt_count <= 48ull * kThreads * 8) fin_base = std::min(fin_base, 48);
  // With several layers the threads visit their candidates four times; as many CTAs as keep those candidates
  // (about twice the entries) in the threads' registers, eight each, save the re-reads.
  int fin_want = (int)(a.pkt_count / 4096);
  if (c->cfg.num_segments > 1) fin_want = (int)((2ull * a.pkt_count + kThreads * 8 - 1) / (kThreads * 8));
  const int fin_grid = std::min(c->finalize_max[MODE], std::max(fin_base, fin_want));
  a.workers = (uint32_t)fin_grid;
  a.packet_format = packet_format_of(c);
  if (c->cfg.flags & DGS_TEST_STALLED_BARRIER) {
    a.phantom_workers = 1;
    a.spin_limit = 4096;
  }
  a.seq = ++c->select_seq;
  a.L_in = single_pass ? c->L_next(KIND, (uint32_t)row) : ws.L_safe;
  task.stream = stream_id;
  if (single_pass && (uint32_t)row != worker) task.reads.push_back(R.ROW(KIND, (uint32_t)row));
  if (a.speculate) task.writes.push_back(R.ROW(KIND, worker));
  task.writes.push_back(R.SCR(KIND, set));
  int rc = task_begin(c, task);
  if (rc != DGS_OK) return rc;
  if (MODE == kPull) {
    rc = catch_up_launch(c, worker, st);
    if (rc != DGS_OK) return rc;
  }
  if (!single_pass) {
    // nothing to go by: histogram of the whole input first, its bounds cannot fail
    TimedLaunch t(c, st, MODE == kPull ? DGS_KERNEL_TWO_PASS_PULL : DGS_KERNEL_TWO_PASS_PUSH);
    k_hist_all<MODE><<<c->hist_grid[MODE], kThreads, 0, st>>>(ws, a);
    DGS_CUDA(c, cudaGetLastError());
    const int pick_grid = (int)std::min<uint32_t>(c->cfg.num_segments, 1024u);
    k_pick_lower<MODE><<<pick_grid, kThreads, 0, st>>>(ws);
    DGS_CUDA(c, cudaGetLastError());
    c->launches += 2;
  }
  {
    TimedLaunch t(c, st, MODE == kPull ? DGS_KERNEL_STREAM_PULL : DGS_KERNEL_STREAM_PUSH);
    // A pull in a context with several workers shares the GPU with the push passes of later events and reads
    // only a small part of D_w: it takes the form of the pass that holds no ring of stages.
    if (MODE == kPull && use_light_pull(c))
      k_pull_light<<<c->stream_grid[MODE], kThreads, 0, st>>>(ws, a);
    else
      k_stream<MODE><<<c->stream_grid[MODE], kThreads, StreamRing<MODE>::kBytes, st>>>(ws, a);
    DGS_CUDA(c, cudaGetLastError());
    c->launches += 1;
  }
  {
    // cooperative launch: the CTAs synchronise among themselves, so all must be resident
    TimedLaunch t(c, st, MODE == kPull ? DGS_KERNEL_FINALIZE_PULL : DGS_KERNEL_FINALIZE_PUSH);
    void* args[] = {(void*)&ws, (void*)&a};
    DGS_CUDA(c, cudaLaunchCooperativeKernel((const void*)k_finalize<MODE>, dim3(fin_grid), dim3(kThreads), args,
                                            finalize_dyn_bytes(c->cfg.num_segments), st));
    c->launches += 1;
  }
  rc = task_end(c, task);
  if (rc != DGS_OK) return rc;
  c->kind_seq[KIND] += 1;
  if (a.speculate) {
    c->row_valid[KIND][worker] = 1;
    c->row_time[KIND][worker] = c->kind_seq[KIND];
    c->row_age[KIND][worker] = age;
  }
  return DGS_OK;
}

template <int MODE>
int occupancy_grids(dgs_ctx* c, int sms) {
  int occ = 0;
  DGS_CUDA(c, cudaFuncSetAttribute(k_stream<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   StreamRing<MODE>::kBytes));
  DGS_CUDA(c, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_stream<MODE>, kThreads,
                                                            StreamRing<MODE>::kBytes));
  if (occ < 1) occ = 1;
  c->stream_grid[MODE] = std::min(sms * occ, kMaxGrid);
  // With several workers a pull's stream pass shares the GPU with the push passes of later events, and
  // what counts is how few SM resources it holds, not how fast it is alone: one CTA per SM (its ranges
  // are balanced by the plan that finalize leaves behind).  A context with one worker selects alone.
  if (MODE == kPull && c->cfg.num_workers > 1) c->stream_grid[MODE] = std::min(c->stream_grid[MODE], sms);
  DGS_CUDA(c, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_hist_all<MODE>, kThreads, 0));
  if (occ < 1) occ = 1;
  c->hist_grid[MODE] = std::min(sms * occ, kMaxGrid);
  DGS_CUDA(c, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_finalize<MODE>, kThreads,
                                                            finalize_dyn_bytes(c->cfg.num_segments)));
  if (occ < 1) {
    c->last_cuda = (int)cudaErrorCooperativeLaunchTooLarge;
    c->broken = true;
    return DGS_ECUDA;
  }
  c->finalize_max[MODE] = std::min(sms * occ, kMaxWorkers);
  c->finalize_grid[MODE] = std::min(c->finalize_max[MODE], kFinalizeWorkers);
  return DGS_OK;
}

void destroy_ctx(dgs_ctx* c) {
  for (int i = 0; i < kNumStreams; ++i) {
    if (c->st[i] && (i == 0 || c->st[i] != c->st[0])) cudaStreamDestroy(c->st[i]);
    if (c->ev_tail[i]) cudaEventDestroy(c->ev_tail[i]);
  }
  if (c->h_chunks) cudaFreeHost(c->h_chunks);
  if (c->ev_in) cudaEventDestroy(c->ev_in);
  for (int i = 0; i < kNumStreams; ++i)
    for (cudaEvent_t e : c->ev_ring[i]) cudaEventDestroy(e);
  for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  c->magic = 0;
  delete c;
}

}  // namespace

extern "C" {

const char* dgs_error_string(int err) {
  switch (err) {
    case DGS_OK: return "ok";
    case DGS_EINVAL: return "invalid argument";
    case DGS_ENOMEM: return "arena too small";
    case DGS_ECUDA: return "CUDA runtime error";
    case DGS_ETIMEOUT: return "bounded device wait expired";
    case DGS_ESTATE: return "context freed or unusable";
    case DGS_ELIMIT: return "size beyond the fixed capacity of the static scratch";
  }
  return "unknown error";
}

int dgs_arena_bytes(const dgs_config* cfg, uint64_t* out_bytes) {
  if (!out_bytes) return DGS_EINVAL;
  const int rc = check_config(cfg);
  if (rc != DGS_OK) return rc;
  Layout L;
  make_layout(cfg, &L);
  *out_bytes = L.total;
  return DGS_OK;
}

int dgs_init(const dgs_config* cfg, dgs_ctx** out) {
  if (!out) return DGS_EINVAL;
  *out = nullptr;
  int rc = check_config(cfg);
  if (rc != DGS_OK) return rc;
  if (!cfg->theta0 || !cfg->arena) return DGS_EINVAL;
  if ((reinterpret_cast<uintptr_t>(cfg->arena) % kAlign) != 0) return DGS_EINVAL;
  dgs_ctx* c = new (std::nothrow) dgs_ctx();
  if (!c) return DGS_ENOMEM;
  c->magic = kMagic;
  c->cfg = *cfg;
  c->segments.assign(cfg->segments, cfg->segments + cfg->num_segments);
  c->cfg.segments = c->segments.data();
  make_layout(&c->cfg, &c->lay);
  for (int i = 0; i < kNumStreams; ++i) {
    c->st[i] = nullptr;
    c->ev_tail[i] = nullptr;
    c->forked[i] = false;
  }
  c->ev_in = nullptr;
  c->task_seq = 0;
  for (int i = 0; i < kNumStreams; ++i) {
    c->ev_next[i] = 0;
    for (int j = 0; j < kNumStreams; ++j) c->waited_seq[i][j] = 0;
  }
  c->pull_count = c->event_count = c->var_count = 0;
  c->log_head = 0;
  c->last_ranges = 0;
  c->cur_gen = 0;
  c->gen_last[0] = c->gen_last[1] = -1;
  c->applied.assign(cfg->num_workers, 0);
  c->kind_seq[0] = c->kind_seq[1] = 0;
  c->res.assign(ResIds{cfg->num_workers}.count(), dgs_ctx::Res());
  if (c->lay.total > cfg->arena_bytes) {
    delete c;
    return DGS_ENOMEM;
  }
  c->base = static_cast<char*>(cfg->arena);
  c->user = static_cast<cudaStream_t>(cfg->stream);
  c->push_count = 0;
  c->inv_m = 1.0f / cfg->momentum;  // one IEEE division; the kernels multiply by this constant
  c->timestamp = 0;
  c->select_seq = 0;
  c->launches = 0;
  c->last_cuda = 0;
  c->broken = false;
  c->timing = false;
  for (int i = 0; i < DGS_NUM_KERNELS; ++i) {
    c->time_ms[i] = 0.0;
    c->time_count[i] = 0;
  }
  for (int k = 0; k < 2; ++k) {
    c->row_valid[k].assign(cfg->num_workers, 0);
    c->row_time[k].assign(cfg->num_workers, 0);
    c->row_age[k].assign(cfg->num_workers, 0);
  }
  c->pushes.assign(cfg->num_workers, 0);
  c->prev.assign(cfg->num_workers, -1);

  auto fail = [&](int code) {
    destroy_ctx(c);
    return code;
  };
#define INIT_CUDA(call)                         \
  do {                                          \
    cudaError_t e_ = (call);                    \
    if (e_ != cudaSuccess) return fail(DGS_ECUDA); \
  } while (0)

  int dev = 0, sms = 0, coop = 0;
  INIT_CUDA(cudaGetDevice(&dev));
  INIT_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  INIT_CUDA(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
  if (!coop) return fail(DGS_ECUDA);
  c->sms = sms;
  c->multi_worker = cfg->num_workers > 1;
  c->h_chunks = nullptr;
  c->seen_chunks[0] = c->seen_chunks[1] = 0;
  c->light_now = false;
  if (c->multi_worker) {
    INIT_CUDA(cudaHostAlloc(reinterpret_cast<void**>(&c->h_chunks), 2 * sizeof(unsigned long long), cudaHostAllocDefault));
    c->h_chunks[0] = c->h_chunks[1] = 0;
  }
  if (occupancy_grids<kPushSam>(c, sms) != DGS_OK || occupancy_grids<kPushResidual>(c, sms) != DGS_OK ||
      occupancy_grids<kPull>(c, sms) != DGS_OK)
    return fail(DGS_ECUDA);
  int prio_low = 0, prio_high = 0;
  INIT_CUDA(cudaDeviceGetStreamPriorityRange(&prio_low, &prio_high));
  for (int i = 0; i < kNumStreams; ++i) {
    // The push passes move most of the bytes and fill every SM; the short kernels of the server side sit on
    // the longer chain (apply -> catch-up -> pull), so their blocks go first whenever an SM has room.
    const int prio = i < kStApply ? prio_low : prio_high;
    if (i > 0 && (cfg->flags & DGS_SINGLE_STREAM))
      c->st[i] = c->st[0];   // every step on one stream: kernels run one after the other, in call order
    else
      INIT_CUDA(cudaStreamCreateWithPriority(&c->st[i], cudaStreamNonBlocking, prio));
    INIT_CUDA(cudaEventCreateWithFlags(&c->ev_tail[i], cudaEventDisableTiming));
  }
  INIT_CUDA(cudaEventCreateWithFlags(&c->ev_in, cudaEventDisableTiming));
  for (int s = 0; s < kNumStreams; ++s)
    for (int i = 0; i < 256; ++i) {
      cudaEvent_t e;
      INIT_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
      c->ev_ring[s].push_back(e);
    }

  const Layout& L = c->lay;
  const uint64_t N = cfg->num_workers, vec = L.n_pad * 4;
  std::vector<Tile> tiles;
  std::vector<SegDesc> segs;
  tiles.reserve(L.num_tiles);
  build_tiles(&c->cfg, &tiles, &segs);
  if (tiles.size() != L.num_tiles) return fail(DGS_EINVAL);
  cudaStream_t st = c->user;
  // state: u = 0, D = 0 (initialisation lines of Algorithm 3 and Algorithm 2), theta = theta_0
  INIT_CUDA(cudaMemsetAsync(c->at<char>(L.u), 0, vec * (N + kPushSets), st));
  INIT_CUDA(cudaMemsetAsync(c->at<char>(L.D), 0, vec * N, st));
  INIT_CUDA(cudaMemsetAsync(c->at<char>(L.theta), 0, vec, st));
  INIT_CUDA(cudaMemcpyAsync(c->at<char>(L.theta), cfg->theta0, cfg->n * 4, cudaMemcpyDeviceToDevice, st));
  if (cfg->flags & DGS_KEEP_LOCAL_MODEL) {
    INIT_CUDA(cudaMemsetAsync(c->at<char>(L.theta_local), 0, vec * N, st));
    for (uint32_t q = 0; q < N; ++q)
      INIT_CUDA(cudaMemcpyAsync(c->theta_local_buf(q), cfg->theta0, cfg->n * 4, cudaMemcpyDeviceToDevice, st));
  }
  // scratch that kernels expect to find cleared, and the static tables
  for (int k = 0; k < kAllSets; ++k) {
    const ScratchLayout& sc = L.sc[k];
    INIT_CUDA(cudaMemsetAsync(c->at<char>(sc.zero_begin), 0, sc.zero_end - sc.zero_begin, st));
    INIT_CUDA(cudaMemsetAsync(c->at<char>(sc.part_cands), 0, (uint64_t)kMaxGrid * 4, st));
    INIT_CUDA(cudaMemsetAsync(c->at<char>(sc.part_slot0), 0, (uint64_t)kMaxGrid * 4, st));
    INIT_CUDA(cudaMemsetAsync(c->at<char>(sc.plan), 0, (uint64_t)(kMaxGrid + 1) * 4, st));   // no plan yet
    INIT_CUDA(cudaMemsetAsync(c->at<char>(sc.part_live), 0, (uint64_t)kMaxGrid * 4, st));
  }
  INIT_CUDA(cudaMemsetAsync(c->at<char>(L.blk_max), 0, N * L.blk_stride * 4, st));   // D = 0
  INIT_CUDA(cudaMemsetAsync(c->at<char>(L.L_next), 0xFF, 2 * N * cfg->num_segments * 4, st));
  INIT_CUDA(cudaMemsetAsync(c->at<char>(L.status), 0, L.total - L.status, st));
  INIT_CUDA(cudaMemcpyAsync(c->at<char>(L.tiles), tiles.data(), tiles.size() * sizeof(Tile), cudaMemcpyHostToDevice, st));
  INIT_CUDA(cudaMemcpyAsync(c->at<char>(L.segs), segs.data(), segs.size() * sizeof(SegDesc), cudaMemcpyHostToDevice, st));
  std::vector<uint32_t> seg_off(cfg->num_segments + 1), seg_tile0(cfg->num_segments);
  for (uint32_t q = 0; q < cfg->num_segments; ++q) {
    seg_off[q] = (uint32_t)cfg->segments[q].offset;
    seg_tile0[q] = segs[q].tile_begin;
  }
  seg_off[cfg->num_segments] = (uint32_t)cfg->n;  // n < 2^32
  INIT_CUDA(cudaMemcpyAsync(c->at<char>(L.seg_off), seg_off.data(), seg_off.size() * 4, cudaMemcpyHostToDevice, st));
  INIT_CUDA(cudaMemcpyAsync(c->at<char>(L.seg_tile0), seg_tile0.data(), seg_tile0.size() * 4, cudaMemcpyHostToDevice, st));
  std::vector<uint32_t> ones(cfg->num_segments, 1u);   // the bound that admits every nonzero value
  INIT_CUDA(cudaMemcpyAsync(c->at<char>(L.L_one), ones.data(), ones.size() * 4, cudaMemcpyHostToDevice, st));
  std::vector<float*> slots(N + kPushSets);
  for (uint32_t q = 0; q < N + kPushSets; ++q) slots[q] = c->u_buf(q);
  INIT_CUDA(cudaMemcpyAsync(c->at<char>(L.u_slots), slots.data(), slots.size() * sizeof(float*), cudaMemcpyHostToDevice, st));
  // the host vectors above go out of scope, and the library's own streams start from a ready arena
  INIT_CUDA(cudaStreamSynchronize(st));
#undef INIT_CUDA

  for (int k = 0; k < kAllSets; ++k) {
    Workspace& w = c->ws[k];
    const ScratchLayout& sc = L.sc[k];
    w.tiles = c->at<Tile>(L.tiles);
    w.segs = c->at<SegDesc>(L.segs);
    w.num_tiles = L.num_tiles;
    w.num_segs = cfg->num_segments;
    w.seg_off = c->at<uint32_t>(L.seg_off);
    w.seg_tile0 = c->at<uint32_t>(L.seg_tile0);
    w.cand_idx = c->at<uint32_t>(sc.cand_idx);
    w.cand_val = c->at<float>(sc.cand_val);
    w.part_cands = c->at<uint32_t>(sc.part_cands);
    w.part_slot0 = c->at<uint32_t>(sc.part_slot0);
    w.plan = c->at<uint32_t>(sc.plan);
    w.part_live = c->at<uint32_t>(sc.part_live);
    w.cta_tot = c->at<uint2>(sc.cta_tot);
    w.seg_start = c->at<uint2>(sc.seg_start);
    w.hist1 = c->at<uint32_t>(sc.hist1);
    w.hist2 = c->at<uint32_t>(sc.hist2);
    w.hist3 = c->at<uint32_t>(sc.hist3);
    w.sel = c->at<SegSel>(sc.sel);
    w.L_safe = c->at<uint32_t>(sc.L_safe);
    w.L_wide = c->at<uint32_t>(sc.L_wide);
    w.sync = c->at<uint32_t>(sc.sync);
    w.status = c->at<int>(L.status);
    w.stats = c->at<unsigned long long>(L.stats);
  }
  c->log.idx = c->at<uint32_t>(L.log_idx);
  c->log.val = c->at<float>(L.log_val);
  c->log.stride = L.log_stride;
  c->log.cap = (uint32_t)L.K[0];
  c->log.ring = L.log_ring;
  c->log.bnd = c->at<uint32_t>(L.log_bnd);
  c->log.pos = c->at<uint32_t>(L.log_pos);
  c->log.ranges = L.log_ranges;
  c->slot_gen.assign(L.log_ring, 0);
  *out = c;
  return DGS_OK;
}

namespace {

int push_impl(dgs_ctx* c, uint32_t worker, const float* grad, dgs_packet* out, bool grad_is_stage) {
  const Layout& L = c->lay;
  const ResIds R{c->cfg.num_workers};
  const int slot = (int)(c->push_count % kPushSlots);
  const int set = (int)(c->push_count % kPushSets);
  const int stream_id = kStW0 + (int)(c->push_count % kWorkerStreams);
  int rc = fork_from_user(c, stream_id);  // the gradient may have been produced on the caller's stream
  if (rc != DGS_OK) return rc;
  SelArgs a;
  std::memset(&a, 0, sizeof(a));
  a.grad = grad;
  a.u_cur_slot = c->u_slot(worker);
  a.u_spare_slot = c->u_slot(c->cfg.num_workers + set);
  a.pkt_idx = c->at<uint32_t>(L.pkt_idx[slot]);
  a.pkt_val = c->at<float>(L.pkt_val[slot]);
  a.pkt_count = (uint32_t)L.K[0];
  a.m = c->cfg.momentum;
  a.lr = c->cfg.lr;
  a.inv_m = c->inv_m;
  Task task;
  task.writes = {R.U(worker), R.SPARE(set), R.PKT(slot)};
  if (grad_is_stage) task.reads.push_back(R.STAGE());
  const uint64_t age = c->pushes[worker];
  rc = (c->cfg.flags & DGS_RESIDUAL_MODE)
           ? launch_select<kPushResidual>(c, a, worker, age, stream_id, set, task)
           : launch_select<kPushSam>(c, a, worker, age, stream_id, set, task);
  if (rc != DGS_OK) return rc;
  c->pushes[worker] += 1;
  c->push_count += 1;
  if (out) {
    out->idx = a.pkt_idx;
    out->val = a.pkt_val;
    out->count = a.pkt_count;
  }
  return DGS_OK;
}

int apply_impl(dgs_ctx* c, uint32_t worker, const dgs_packet* pkt) {
  (void)worker;
  const ResIds R{c->cfg.num_workers};
  const uint32_t N = c->cfg.num_workers;
  // whose packet is it?  one of the push slots: the tracker knows its writer; anything else: the caller's stream
  int slot = -1;
  for (int i = 0; i < kPushSlots; ++i)
    if (pkt->idx == c->at<uint32_t>(c->lay.pkt_idx[i])) slot = i;
  const uint32_t gx = (pkt->count + kThreads - 1) / kThreads;
  if (pkt->count == 0) {
    // nothing to subtract
  } else if (slot >= 0 && pkt->val == c->at<float>(c->lay.pkt_val[slot]) && pkt->count == c->log.cap) {
    // One of the library's own packets (sorted by index, of the fixed size): theta now, the D_q lazily.
    // Its slot of the log still holds the packet filed `ring` applies ago; whoever has not folded that
    // one in yet does so first.
    const uint32_t lslot = (uint32_t)(c->log_head % c->log.ring);
    if (c->log_head >= c->log.ring) {
      const uint64_t oldest = c->log_head - c->log.ring;
      for (uint32_t q = 0; q < N; ++q)
        if (c->applied[q] <= oldest) {
          const int rc = catch_up_now(c, q);
          if (rc != DGS_OK) return rc;
        }
    }
    // The ranges of the log are taken from the first packet filed, again from packet N (velocities have
    // built up by then) and then every few rounds of the workers, so that they follow a drifting
    // distribution.  Packets keep the positions they were filed with: the ranges come in two generations,
    // a packet's slot remembers which one its positions refer to, and a catch-up folds the packets of the
    // older generation before those of the newer one.  A generation is overwritten only when every packet
    // filed under it has left the ring, so nobody has to catch up for the ranges to change.
    const uint64_t period = std::max<uint64_t>(16ull * N, 2ull * c->log.ring);
    const bool new_ranges = c->log_head == 0 || (c->log_head == N && c->last_ranges == 0) ||
                            c->log_head >= c->last_ranges + period;
    if (new_ranges) {
      if (c->log_head > 0) {
        // the other generation is taken over: whoever still has to fold in one of its packets (a worker that
        // stayed away for very long) does so first
        const int other = c->cur_gen ^ 1;
        for (uint32_t q = 0; q < N; ++q)
          if ((int64_t)c->applied[q] <= c->gen_last[other]) {
            const int rc = catch_up_now(c, q);
            if (rc != DGS_OK) return rc;
          }
        c->cur_gen = other;
      }
      c->last_ranges = c->log_head;
    }
    c->gen_last[c->cur_gen] = (int64_t)c->log_head;
    c->slot_gen[lslot] = (uint8_t)c->cur_gen;
    PacketLog lg = c->log;
    lg.bnd = c->log.bnd + (size_t)c->cur_gen * c->log.ranges;
    Task t;
    t.stream = kStApply;
    t.reads.push_back(R.PKT(slot));
    t.writes = {R.THETA(), R.LOG(lslot)};
    if (new_ranges) t.writes.push_back(R.RANGES(c->cur_gen));
    else t.reads.push_back(R.RANGES(c->cur_gen));
    int rc = task_begin(c, t);
    if (rc != DGS_OK) return rc;
    {
      TimedLaunch tl(c, c->st[kStApply], DGS_KERNEL_SCATTER);
      if (new_ranges) {
        k_log_ranges<<<(c->log.ranges + kThreads - 1) / kThreads, kThreads, 0, c->st[kStApply]>>>(pkt->idx, lg);
        DGS_CUDA(c, cudaGetLastError());
        c->launches += 1;
      }
      const uint32_t pos_ctas = (c->log.ranges + 1 + kThreads - 1) / kThreads;
      k_apply_log<<<gx + pos_ctas, kThreads, 0, c->st[kStApply]>>>(pkt->idx, pkt->val, pkt->count,
                                                                   c->at<float>(c->lay.theta), c->cfg.n,
                                                                   c->ws[0].status, lg, lslot, gx);
      DGS_CUDA(c, cudaGetLastError());
      c->launches += 1;
    }
    rc = task_end(c, t);
    if (rc != DGS_OK) return rc;
    c->log_head += 1;
  } else {
    // Any other packet: bring every D_q up to date, then subtract from theta and all of them at once.
    for (uint32_t q = 0; q < N; ++q) {
      const int rc = catch_up_now(c, q);
      if (rc != DGS_OK) return rc;
    }
    Task t;
    t.stream = kStApply;
    if (slot >= 0) t.reads.push_back(R.PKT(slot));
    t.writes.push_back(R.THETA());
    for (uint32_t q = 0; q < N; ++q) t.writes.push_back(R.D(q));
    int rc = slot >= 0 ? DGS_OK : fork_from_user(c, kStApply);
    if (rc != DGS_OK) return rc;
    rc = task_begin(c, t);
    if (rc != DGS_OK) return rc;
    {
      TimedLaunch tl(c, c->st[kStApply], DGS_KERNEL_SCATTER);
      k_scatter_sub<<<dim3(gx, N + 1), kThreads, 0, c->st[kStApply]>>>(
          pkt->idx, pkt->val, pkt->count, c->at<float>(c->lay.theta), c->at<float>(c->lay.D), c->lay.n_pad, N,
          c->cfg.n, c->ws[0].status, c->blk_max(0), c->lay.blk_stride);
      DGS_CUDA(c, cudaGetLastError());
      c->launches += 1;
    }
    rc = task_end(c, t);
    if (rc != DGS_OK) return rc;
  }
  c->timestamp += 1;  // t counts updates made to the server parameters
  return DGS_OK;
}

int pull_impl(dgs_ctx* c, uint32_t worker, dgs_packet* out) {
  const Layout& L = c->lay;
  const ResIds R{c->cfg.num_workers};
  const int slot = kPushSlots + (int)(c->pull_count % kPullSlots);
  const int set = (int)(c->pull_count % kPullSets);
  const int stream_id = kStS0 + (int)(c->pull_count % kServerStreams);
  int rc = fork_from_user(c, stream_id);  // the caller may still be reading an older pull packet on its stream
  if (rc != DGS_OK) return rc;
  SelArgs a;
  std::memset(&a, 0, sizeof(a));
  a.D = c->D_buf(worker);
  a.blk_max = c->blk_max(worker);
  a.theta_local = (c->cfg.flags & DGS_KEEP_LOCAL_MODEL) ? c->theta_local_buf(worker) : nullptr;
  a.pkt_idx = c->at<uint32_t>(L.pkt_idx[slot]);
  a.pkt_val = c->at<float>(L.pkt_val[slot]);
  a.pkt_count = (uint32_t)L.K[1];
  a.m = c->cfg.momentum;
  a.lr = c->cfg.lr;
  a.inv_m = c->inv_m;
  Task task;
  task.writes = {R.PKT(slot)};
  catch_up_deps(c, worker, &task);  // D_worker is brought up to date first, on the same stream
  if (a.theta_local) task.writes.push_back(R.TL(worker));
  // packets that entered D_worker since its previous pull
  const uint64_t age = c->timestamp - (c->prev[worker] < 0 ? 0 : (uint64_t)c->prev[worker]);
  rc = launch_select<kPull>(c, a, worker, age, stream_id, set, task);
  if (rc != DGS_OK) return rc;
  rc = report_chunks(c, c->st[stream_id]);
  if (rc != DGS_OK) return rc;
  c->prev[worker] = (int64_t)c->timestamp;
  c->pull_count += 1;
  if (out) {
    out->idx = a.pkt_idx;
    out->val = a.pkt_val;
    out->count = a.pkt_count;
  }
  return DGS_OK;
}

// Pull without secondary compression: catch-up, the pull's stream pass with the bound 1 (every nonzero entry
// becomes a candidate, in index order), then the copy into the packet.  Shares the pulls' streams and scratch sets.
int pull_all_impl(dgs_ctx* c, uint32_t worker, dgs_var_packet* out) {
  const Layout& L = c->lay;
  const ResIds R{c->cfg.num_workers};
  const int vslot = (int)(c->var_count % kVarSlots);
  const int set = (int)(c->pull_count % kPullSets);
  const int stream_id = kStS0 + (int)(c->pull_count % kServerStreams);
  cudaStream_t st = c->st[stream_id];
  int rc = fork_from_user(c, stream_id);  // the caller may still be reading an older packet on its stream
  if (rc != DGS_OK) return rc;
  Workspace& ws = c->ws[kPushSets + set];
  SelArgs a;
  std::memset(&a, 0, sizeof(a));
  a.D = c->D_buf(worker);
  a.blk_max = c->blk_max(worker);
  a.theta_local = (c->cfg.flags & DGS_KEEP_LOCAL_MODEL) ? c->theta_local_buf(worker) : nullptr;
  a.L_in = c->at<uint32_t>(L.L_one);
  a.m = c->cfg.momentum;
  a.lr = c->cfg.lr;
  a.inv_m = c->inv_m;
  Task task;
  task.stream = stream_id;
  task.writes = {R.VPKT(vslot), R.SCR(1, set)};
  catch_up_deps(c, worker, &task);  // D_worker is brought up to date first, on the same stream
  if (a.theta_local) task.writes.push_back(R.TL(worker));
  rc = task_begin(c, task);
  if (rc != DGS_OK) return rc;
  rc = catch_up_launch(c, worker, st);
  if (rc != DGS_OK) return rc;
  {
    TimedLaunch t(c, st, DGS_KERNEL_STREAM_PULL);
    if (use_light_pull(c))
      k_pull_light<<<c->stream_grid[kPull], kThreads, 0, st>>>(ws, a);
    else
      k_stream<kPull><<<c->stream_grid[kPull], kThreads, StreamRing<kPull>::kBytes, st>>>(ws, a);
    DGS_CUDA(c, cudaGetLastError());
    c->launches += 1;
  }
  uint32_t* vi = c->at<uint32_t>(L.var_idx[vslot]);
  float* vv = c->at<float>(L.var_val[vslot]);
  uint32_t* vc = c->at<uint32_t>(L.var_count[vslot]);
  {
    TimedLaunch t(c, st, DGS_KERNEL_FINALIZE_PULL);
    k_emit_all<<<2 * c->sms, kThreads, 0, st>>>(ws, a.D, a.theta_local, a.blk_max, vi, vv, vc, c->cfg.pull_all_capacity,
                                                packet_format_of(c));
    DGS_CUDA(c, cudaGetLastError());
    c->launches += 1;
  }
  rc = task_end(c, task);
  if (rc != DGS_OK) return rc;
  rc = report_chunks(c, st);
  if (rc != DGS_OK) return rc;
  c->prev[worker] = (int64_t)c->timestamp;
  c->pull_count += 1;
  c->var_count += 1;
  if (out) {
    out->idx = vi;
    out->val = vv;
    out->count = vc;
    out->capacity = c->cfg.pull_all_capacity;
  }
  return DGS_OK;
}

}  // namespace

int dgs_worker_pull_all(dgs_ctx* c, uint32_t worker, dgs_var_packet* out) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (worker >= c->cfg.num_workers || c->cfg.pull_all_capacity == 0) return DGS_EINVAL;
  rc = begin_call(c);
  if (rc != DGS_OK) return rc;
  return pull_all_impl(c, worker, out);
}

int dgs_worker_push(dgs_ctx* c, uint32_t worker, const float* grad, dgs_packet* out) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (worker >= c->cfg.num_workers || !grad) return DGS_EINVAL;
  if ((reinterpret_cast<uintptr_t>(grad) % 16) != 0) return DGS_EINVAL;
  rc = begin_call(c);
  if (rc != DGS_OK) return rc;
  return push_impl(c, worker, grad, out, false);
}

int dgs_server_apply(dgs_ctx* c, uint32_t worker, const dgs_packet* pkt) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (worker >= c->cfg.num_workers || !pkt) return DGS_EINVAL;
  if (pkt->count > 0 && (!pkt->idx || !pkt->val)) return DGS_EINVAL;
  rc = begin_call(c);
  if (rc != DGS_OK) return rc;
  return apply_impl(c, worker, pkt);
}

int dgs_worker_pull(dgs_ctx* c, uint32_t worker, dgs_packet* out) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (worker >= c->cfg.num_workers) return DGS_EINVAL;
  rc = begin_call(c);
  if (rc != DGS_OK) return rc;
  return pull_impl(c, worker, out);
}

int dgs_event(dgs_ctx* c, uint32_t worker, const float* grad, dgs_packet* push_out, dgs_packet* pull_out) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (worker >= c->cfg.num_workers || !grad) return DGS_EINVAL;
  if ((reinterpret_cast<uintptr_t>(grad) % 16) != 0) return DGS_EINVAL;
  rc = begin_call(c);
  if (rc != DGS_OK) return rc;
  dgs_packet p, g;
  rc = push_impl(c, worker, grad, &p, false);
  if (rc != DGS_OK) return rc;
  rc = apply_impl(c, worker, &p);
  if (rc != DGS_OK) return rc;
  rc = pull_impl(c, worker, &g);
  if (rc != DGS_OK) return rc;
  if (push_out) *push_out = p;
  if (pull_out) *pull_out = g;
  return DGS_OK;
}

int dgs_flush(dgs_ctx* c) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  for (int i = 0; i < kNumStreams; ++i) {
    DGS_CUDA(c, cudaEventRecord(c->ev_tail[i], c->st[i]));
    DGS_CUDA(c, cudaStreamWaitEvent(c->user, c->ev_tail[i], 0));
  }
  return DGS_OK;
}

int dgs_event_host(dgs_ctx* c, uint32_t worker, const float* grad_host, uint32_t* out_idx, float* out_val) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (!(c->cfg.flags & DGS_HOST_IO) || !grad_host || worker >= c->cfg.num_workers) return DGS_EINVAL;
  rc = begin_call(c);
  if (rc != DGS_OK) return rc;
  const ResIds R{c->cfg.num_workers};
  float* stage = c->at<float>(c->lay.grad_stage);
  {
    // host -> staging buffer, on the stream of the push that will read it
    Task t;
    t.stream = kStW0 + (int)(c->push_count % kWorkerStreams);
    t.writes.push_back(R.STAGE());
    rc = fork_from_user(c, t.stream);
    if (rc != DGS_OK) return rc;
    rc = task_begin(c, t);
    if (rc != DGS_OK) return rc;
    DGS_CUDA(c, cudaMemcpyAsync(stage, grad_host, c->cfg.n * 4, cudaMemcpyHostToDevice, c->st[t.stream]));
    rc = task_end(c, t);
    if (rc != DGS_OK) return rc;
  }
  dgs_packet p, g;
  rc = push_impl(c, worker, stage, &p, true);
  if (rc != DGS_OK) return rc;
  rc = apply_impl(c, worker, &p);
  if (rc != DGS_OK) return rc;
  const int pull_stream = kStS0 + (int)(c->pull_count % kServerStreams);
  rc = pull_impl(c, worker, &g);
  if (rc != DGS_OK) return rc;
  cudaStream_t ps = c->st[pull_stream];
  if (out_idx) DGS_CUDA(c, cudaMemcpyAsync(out_idx, g.idx, (uint64_t)g.count * 4, cudaMemcpyDeviceToHost, ps));
  if (out_val) DGS_CUDA(c, cudaMemcpyAsync(out_val, g.val, (uint64_t)g.count * 4, cudaMemcpyDeviceToHost, ps));
  // the event is complete when its pull is (the pull waited for the apply, the apply for the push),
  // except for the shares of the apply that run on the other server streams
  DGS_CUDA(c, cudaStreamSynchronize(ps));
  for (int i = 0; i < kServerStreams; ++i) DGS_CUDA(c, cudaStreamSynchronize(c->st[kStS0 + i]));
  return DGS_OK;
}

int dgs_state_ptr(dgs_ctx* c, int which, uint32_t worker, const float** out) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (!out) return DGS_EINVAL;
  if (which != DGS_THETA && worker >= c->cfg.num_workers) return DGS_EINVAL;
  switch (which) {
    case DGS_THETA: *out = c->at<float>(c->lay.theta); break;
    case DGS_D:
      rc = catch_up_now(c, worker);
      if (rc != DGS_OK) return rc;
      *out = c->D_buf(worker);
      break;
    case DGS_THETA_LOCAL:
      if (!(c->cfg.flags & DGS_KEEP_LOCAL_MODEL)) return DGS_EINVAL;
      *out = c->theta_local_buf(worker);
      break;
    case DGS_U: {
      float* p = nullptr;
      rc = sync_all(c);
      if (rc != DGS_OK) return rc;
      DGS_CUDA(c, cudaMemcpy(&p, c->u_slot(worker), sizeof(p), cudaMemcpyDeviceToHost));
      *out = p;
      return DGS_OK;
    }
    default: return DGS_EINVAL;
  }
  return sync_all(c);
}

int dgs_state_load(dgs_ctx* c, int which, uint32_t worker, const float* src) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (!src) return DGS_EINVAL;
  const float* dst = nullptr;
  rc = dgs_state_ptr(c, which, worker, &dst);  // waits for all work in flight
  if (rc != DGS_OK) return rc;
  rc = begin_call(c);
  if (rc != DGS_OK) return rc;
  const ResIds R{c->cfg.num_workers};
  Task t;
  t.stream = kStApply;
  t.writes.push_back(which == DGS_THETA ? R.THETA()
                     : which == DGS_U   ? R.U(worker)
                     : which == DGS_D   ? R.D(worker)
                                        : R.TL(worker));
  rc = fork_from_user(c, t.stream);
  if (rc != DGS_OK) return rc;
  rc = task_begin(c, t);
  if (rc != DGS_OK) return rc;
  DGS_CUDA(c, cudaMemcpyAsync(const_cast<float*>(dst), src, c->cfg.n * 4, cudaMemcpyDeviceToDevice, c->st[t.stream]));
  if (which == DGS_D)   // nothing is known about the new contents: every block may hold anything
    DGS_CUDA(c, cudaMemsetAsync(c->blk_max(worker), 0xFF, c->lay.blk_stride * 4, c->st[t.stream]));
  return task_end(c, t);
}

int dgs_status(dgs_ctx* c, int* device_status) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (!device_status) return DGS_EINVAL;
  rc = sync_all(c);
  if (rc != DGS_OK) return rc;
  DGS_CUDA(c, cudaMemcpy(device_status, c->ws[0].status, 4, cudaMemcpyDeviceToHost));
  return DGS_OK;
}

int dgs_stats(dgs_ctx* c, uint64_t out[4]) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (!out) return DGS_EINVAL;
  unsigned long long s[4] = {0, 0, 0, 0};
  rc = sync_all(c);
  if (rc != DGS_OK) return rc;
  DGS_CUDA(c, cudaMemcpy(s, c->ws[0].stats, sizeof(s), cudaMemcpyDeviceToHost));
  out[0] = s[0];
  out[1] = s[1];
  out[2] = c->timestamp;
  out[3] = s[2];
  return DGS_OK;
}

int dgs_pull_read_stats(dgs_ctx* c, uint64_t out[2]) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (!out) return DGS_EINVAL;
  unsigned long long s[2] = {0, 0};
  rc = sync_all(c);
  if (rc != DGS_OK) return rc;
  DGS_CUDA(c, cudaMemcpy(s, c->ws[0].stats + 3, sizeof(s), cudaMemcpyDeviceToHost));
  out[0] = s[0];
  out[1] = s[1];
  return DGS_OK;
}

int dgs_prev(dgs_ctx* c, uint32_t worker, int64_t* out) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (!out || worker >= c->cfg.num_workers) return DGS_EINVAL;
  *out = c->prev[worker];
  return DGS_OK;
}

int dgs_launch_count(dgs_ctx* c, uint64_t* out) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (!out) return DGS_EINVAL;
  *out = c->launches;
  return DGS_OK;
}

int dgs_timing_enable(dgs_ctx* c, int on) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  c->timing = on != 0;
  return DGS_OK;
}

int dgs_timing_read(dgs_ctx* c, double ms[DGS_NUM_KERNELS], uint64_t count[DGS_NUM_KERNELS]) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (!ms || !count) return DGS_EINVAL;
  rc = sync_all(c);
  if (rc != DGS_OK) return rc;
  for (size_t i = 0; i < c->ev_kernel.size(); ++i) {
    float t = 0.f;
    DGS_CUDA(c, cudaEventElapsedTime(&t, c->ev_pool[2 * i], c->ev_pool[2 * i + 1]));
    c->time_ms[c->ev_kernel[i]] += t;
    c->time_count[c->ev_kernel[i]] += 1;
  }
  c->ev_kernel.clear();
  c->ev_stream.clear();
  for (int i = 0; i < DGS_NUM_KERNELS; ++i) {
    ms[i] = c->time_ms[i];
    count[i] = c->time_count[i];
    c->time_ms[i] = 0.0;
    c->time_count[i] = 0;
  }
  return DGS_OK;
}

int dgs_timing_trace(dgs_ctx* c, uint32_t cap, float* start_ms, float* stop_ms, int32_t* kernel, int32_t* stream,
                     uint32_t* count) {
  int rc = live(c);
  if (rc != DGS_OK) return rc;
  if (!start_ms || !stop_ms || !kernel || !stream || !count) return DGS_EINVAL;
  rc = sync_all(c);
  if (rc != DGS_OK) return rc;
  const size_t m = std::min<size_t>(cap, c->ev_kernel.size());
  for (size_t i = 0; i < m; ++i) {
    DGS_CUDA(c, cudaEventElapsedTime(start_ms + i, c->ev_pool[0], c->ev_pool[2 * i]));
    DGS_CUDA(c, cudaEventElapsedTime(stop_ms + i, c->ev_pool[0], c->ev_pool[2 * i + 1]));
    kernel[i] = c->ev_kernel[i];
    stream[i] = c->ev_stream[i];
  }
  *count = (uint32_t)m;
  c->ev_kernel.clear();
  c->ev_stream.clear();
  return DGS_OK;
}

int dgs_hardware_queues(int* needed, int* configured) {
  if (needed) *needed = kNumStreams + 1;
  if (configured) {
    int v = 8;   // the driver's default
    if (const char* e = std::getenv("CUDA_DEVICE_MAX_CONNECTIONS")) {
      char* endp = nullptr;
      const long x = std::strtol(e, &endp, 10);
      if (endp != e && x >= 1 && x <= 32) v = (int)x;
    }
    *configured = v;
  }
  return DGS_OK;
}

int dgs_last_cuda_error(dgs_ctx* c) {
  if (!c || c->magic != kMagic) return 0;
  return c->last_cuda;
}

int dgs_free(dgs_ctx* c) {
  if (!c || c->magic != kMagic) return DGS_ESTATE;
  for (int i = 0; i < kNumStreams; ++i) cudaStreamSynchronize(c->st[i]);
  cudaStreamSynchronize(c->user);
  destroy_ctx(c);
  return DGS_OK;
}

}  // extern "C"

// ---- top-k + encode with all scratch in the device image (dgs_topk_encode_static) --------
namespace {

constexpr uint32_t kStaticMaxN = DGS_STATIC_MAX_N;
constexpr uint32_t kStaticMaxTiles = kStaticMaxN / kWarpTile;  // one layer starting at 0: no ragged head

struct StaticScratch {
  float x[kStaticMaxN];            // private copy of the input (the selection clears what it sends)
  uint32_t cand_idx[kStaticMaxN];
  float cand_val[kStaticMaxN];
  Tile tiles[kStaticMaxTiles];
  uint32_t part_cands[kMaxGrid];
  uint32_t part_slot0[kMaxGrid];
  uint2 cta_tot[kMaxWorkers];
  uint2 seg_start[1];
  uint32_t hist1[kBins1];
  uint32_t hist2[kBins2];
  uint32_t hist3[kBins3];
  SegDesc seg;
  SegSel sel;
  uint32_t seg_off[2];
  uint32_t seg_tile0[1];
  uint32_t L_safe[1];
  uint32_t L_wide[1];
  uint32_t L_next[1];
  uint32_t sync[kNumSyncWords];
  int status;
  unsigned long long stats[kNumStats];   // the kernels index words 0 .. 4
};
static_assert(sizeof(((StaticScratch*)nullptr)->stats) == kNumStats * sizeof(unsigned long long),
              "the static scratch must hold every counter a Workspace has");

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress,
// never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

// Tables of a one-layer problem and everything that has to start at zero.
__global__ void k_static_prepare(StaticScratch* sc, uint32_t n, uint32_t k, uint32_t num_tiles) {
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < num_tiles) {
    Tile t;
    t.start = i * kWarpTile;
    t.len = (uint16_t)min((uint32_t)kWarpTile, n - i * kWarpTile);
    t.seg = 0;
    sc->tiles[i] = t;
  }
  if (i < kBins1) sc->hist1[i] = 0;
  if (i < kBins2) sc->hist2[i] = 0;
  if (i < kBins3) sc->hist3[i] = 0;
  if (i < kMaxGrid) {
    sc->part_cands[i] = 0;
    sc->part_slot0[i] = 0;
  }
  if (i == 0) {
    sc->seg.tile_begin = 0;
    sc->seg.tile_end = num_tiles;
    sc->seg.k[0] = sc->seg.k[1] = k;
    sc->seg.pkt_off[0] = sc->seg.pkt_off[1] = 0;
    sc->seg_off[0] = 0;
    sc->seg_off[1] = n;
    sc->seg_tile0[0] = 0;
    sc->sync[kBarCount] = 0;
    sc->sync[kFail] = 0;
    sc->status = 0;
  }
}

struct StaticDevice {
  bool ready = false;
  StaticScratch* scratch = nullptr;  // device address of g_static_scratch on this device
  int stream_grid = 0, hist_grid = 0, finalize_grid = 0;
};
constexpr int kMaxDevices = 64;
StaticDevice g_static_dev[kMaxDevices];
std::mutex g_static_mu;

// Once per device, with that device current.
int static_setup(int dev, StaticDevice** out) {
  std::lock_guard<std::mutex> lock(g_static_mu);
  StaticDevice& d = g_static_dev[dev];
  if (!d.ready) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return DGS_ECUDA;
    int sms = 0, coop = 0, occ = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return DGS_ECUDA;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return DGS_ECUDA;
    if (cudaFuncSetAttribute(k_stream<kPull>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             StreamRing<kPull>::kBytes) != cudaSuccess)
      return DGS_ECUDA;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_stream<kPull>, kThreads, StreamRing<kPull>::kBytes) !=
        cudaSuccess)
      return DGS_ECUDA;
    d.stream_grid = std::min(sms * std::max(occ, 1), kMaxGrid);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_hist_all<kPull>, kThreads, 0) != cudaSuccess) return DGS_ECUDA;
    d.hist_grid = std::min(sms * std::max(occ, 1), kMaxGrid);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_finalize<kPull>, kThreads, finalize_dyn_bytes(1)) !=
            cudaSuccess ||
        occ < 1)
      return DGS_ECUDA;
    d.finalize_grid = std::min(std::min(sms * occ, kMaxWorkers), kFinalizeWorkers);
    d.scratch = static_cast<StaticScratch*>(p);
    d.ready = true;
  }
  *out = &d;
  return DGS_OK;
}

}  // namespace

extern "C" int dgs_topk_encode_static(const float* x, uint32_t n, uint32_t k, uint32_t* out_idx, float* out_val,
                                      void* stream) {
  if (!x || !out_idx || !out_val || n == 0 || k == 0 || k > n) return DGS_EINVAL;
  if (n > kStaticMaxN) return DGS_ELIMIT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DGS_ECUDA;
  StaticDevice* d = nullptr;
  const int rc = static_setup(dev, &d);
  if (rc != DGS_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  StaticScratch* sc = d->scratch;  // device address: only ever dereferenced by kernels
  const uint32_t num_tiles = (n + kWarpTile - 1) / kWarpTile;

  Workspace ws;
  ws.tiles = sc->tiles;
  ws.segs = &sc->seg;
  ws.num_tiles = num_tiles;
  ws.num_segs = 1;
  ws.cand_idx = sc->cand_idx;
  ws.cand_val = sc->cand_val;
  ws.part_cands = sc->part_cands;
  ws.part_slot0 = sc->part_slot0;
  ws.plan = nullptr;
  ws.part_live = nullptr;
  ws.seg_off = sc->seg_off;
  ws.seg_tile0 = sc->seg_tile0;
  ws.cta_tot = sc->cta_tot;
  ws.seg_start = sc->seg_start;
  ws.hist1 = sc->hist1;
  ws.hist2 = sc->hist2;
  ws.hist3 = sc->hist3;
  ws.sel = &sc->sel;
  ws.L_safe = sc->L_safe;
  ws.L_wide = sc->L_wide;
  ws.sync = sc->sync;
  ws.status = &sc->status;
  ws.stats = sc->stats;

  SelArgs a;
  std::memset(&a, 0, sizeof(a));
  a.D = sc->x;
  a.L_in = sc->L_safe;
  a.L_next = sc->L_next;
  a.pkt_idx = out_idx;
  a.pkt_val = out_val;
  a.pkt_count = k;
  a.m = 1.0f;
  a.inv_m = 1.0f;
  a.force_two_pass = 1;
  a.speculate = 0;
  a.workers = (uint32_t)d->finalize_grid;
  a.seq = 0;

  if (cudaMemcpyAsync(sc->x, x, (size_t)n * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return DGS_ECUDA;
  // every launch is checked before the next one is enqueued: a kernel that did not start must not be
  // followed by kernels that count on what it clears (peek: an earlier error of the caller's stays the caller's)
  const uint32_t prep_items = std::max<uint32_t>(num_tiles, kBins1);
  k_static_prepare<<<(prep_items + kThreads - 1) / kThreads, kThreads, 0, st>>>(sc, n, k, num_tiles);
  if (cudaPeekAtLastError() != cudaSuccess) return DGS_ECUDA;
  k_hist_all<kPull><<<d->hist_grid, kThreads, 0, st>>>(ws, a);
  if (cudaPeekAtLastError() != cudaSuccess) return DGS_ECUDA;
  k_pick_lower<kPull><<<1, kThreads, 0, st>>>(ws);
  if (cudaPeekAtLastError() != cudaSuccess) return DGS_ECUDA;
  k_stream<kPull><<<d->stream_grid, kThreads, StreamRing<kPull>::kBytes, st>>>(ws, a);
  if (cudaPeekAtLastError() != cudaSuccess) return DGS_ECUDA;
  void* args[] = {(void*)&ws, (void*)&a};
  if (cudaLaunchCooperativeKernel((const void*)k_finalize<kPull>, dim3(d->finalize_grid), dim3(kThreads), args,
                                  finalize_dyn_bytes(1), st) != cudaSuccess)
    return DGS_ECUDA;
  return DGS_OK;
}

extern "C" int dgs_topk_encode_static_status(void* stream, int* device_status) {
  if (!device_status) return DGS_EINVAL;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DGS_ECUDA;
  StaticDevice* d = nullptr;
  const int rc = static_setup(dev, &d);
  if (rc != DGS_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int word = 0;
  if (cudaMemcpyAsync(&word, &d->scratch->status, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return DGS_ECUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return DGS_ECUDA;
  *device_status = word;
  return DGS_OK;
}
