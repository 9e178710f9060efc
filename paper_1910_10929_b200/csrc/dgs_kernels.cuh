// Device code of the DGS push / apply / pull loop for sm_100a.
//
// Selection scheme (used for the worker's top-k of the velocity, Algorithm 3, and
// for the server's top-k of the model difference, Algorithm 2 / Eq. 6a):
//
//   stream pass   one read of the input by all SMs.  Every element whose magnitude
//                 key is at least a per-layer lower bound L becomes a "candidate".
//                 A warp handles one tile of 512 elements at a time and appends the
//                 tile's candidates, in index order, as one "run" to its CTA's region
//                 of the candidate buffer.  Everything below L is final at once (the
//                 push writes t*(1/m) there).
//   finalize      one small kernel (a few dozen co-resident CTAs with a barrier of
//                 their own) over the candidates only: three radix levels (11+10+10
//                 key bits) give the exact k-th largest key T and the number r of
//                 entries equal to T that still fit; a count / scan / emit writes the
//                 packet in index order.
//
// L is a guess carried over from an earlier selection of the same kind on that layer
// (the host picks the most recent one made in a comparable state).  The guess is
// checked exactly (a layer needs at least k candidates).  With nothing to carry
// over, a histogram pass over the entire input comes first and gives a bound that
// cannot fail; when a guess fails, finalize redoes both passes itself.  The result
// never depends on the guess.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dgs {

constexpr int kWarpTile = 512;      // elements per tile (one warp, 4 x float4 per lane)
constexpr int kVecIters = 4;
constexpr int kThreads = 256;       // threads per CTA in every kernel here
constexpr int kWarps = kThreads / 32;
constexpr int kBins1 = 2048;        // key bits 30..20
constexpr int kBins2 = 1024;        // key bits 19..10
constexpr int kBins3 = 1024;        // key bits  9..0
constexpr uint32_t kFull = 0xFFFFFFFFu;
constexpr uint32_t kSpecFactor = 3; // aim for max(3k, k+64) candidates next time
constexpr uint32_t kSpecSlack = 64;
constexpr int kMaxGrid = 1024;      // upper bound on the grid of a stream pass (= parts of the candidate buffer)
constexpr int kMaxWorkers = 128;    // upper bound on the grid of finalize
constexpr uint32_t kSpinLimit = 1u << 22;  // bounded waits: give up and report after this many polls
constexpr int kStatusTimeout = -4;  // = DGS_ETIMEOUT

enum Mode : int { kPushSam = 0, kPushResidual = 1, kPull = 2 };

struct Tile {          // a run of <= kWarpTile elements inside one layer
  uint32_t start;
  uint16_t len;
  uint16_t seg;
};

struct SegDesc {
  uint32_t tile_begin, tile_end;  // tiles of this layer
  uint32_t k[2];                  // [0] push, [1] pull
  uint32_t pkt_off[2];            // exclusive prefix of k over layers
};

struct SegSel {        // per-layer selection state of the selection in flight
  uint32_t prefix;     // key bits fixed so far
  uint32_t krem;       // entries still to take at or below the fixed prefix
  uint32_t T;          // k-th largest key
  uint32_t r;          // entries with key == T that are taken (lowest indices)
};

// word indices in Workspace::sync
enum SyncWord : int { kBarCount = 0, kBarGen = 1, kDecision = 2, kFail = 3, kParts = 4, kNumSyncWords = 8 };

struct Workspace {
  const Tile* tiles;
  const SegDesc* segs;
  uint32_t num_tiles, num_segs;
  // candidates: part p (CTA p of the grid that ran the stream pass, `parts` CTAs) owns the slots
  // starting at the first element of its first tile
  uint32_t* cand_idx;     // [n]
  float* cand_val;        // [n]
  uint32_t* part_cands;   // [kMaxGrid] candidates written by each part
  uint32_t* part_slot0;   // [kMaxGrid] first slot of each part
  const uint32_t* seg_off;   // [S+1] first element of each layer, and n
  const uint32_t* seg_tile0; // [S]   first tile of each layer
  uint2* tile_sel;        // [num_tiles] (#key > T, #key == T) per tile; all zero between selections
  uint2* tile_pre;        // [num_tiles] exclusive prefix of tile_sel inside the scanning CTA's chunk
  uint2* cta_tot;         // [kMaxWorkers]
  uint32_t* hist1;        // [S][kBins1]
  uint32_t* hist2;        // [S][kBins2]
  uint32_t* hist3;        // [S][kBins3]
  SegSel* sel;            // [S]
  uint32_t* L_safe;       // [S] bound from the whole-input histogram (two-pass route)
  uint32_t* sync;         // [kNumSyncWords]
  int* status;            // sticky device status word
  unsigned long long* stats;  // [0] single-pass selections, [1] two-pass selections, [2] candidates seen
};

struct SelArgs {
  const float* grad;      // push: f32[n]
  float** u_cur_slot;     // push: device slot holding the worker's velocity pointer
  float** u_spare_slot;   // push: device slot holding the spare buffer pointer
  float* D;               // pull: D_w
  float* theta_local;     // pull: theta_w or null
  const uint32_t* L_in;   // [S] lower bounds guessed for this selection (single-pass route)
  uint32_t* L_next;       // [S] receives the bounds this selection suggests for a later, similar one
  uint32_t* pkt_idx;
  float* pkt_val;
  uint32_t pkt_count;
  float m, lr, inv_m;
  int force_two_pass;
  int speculate;          // 0: never carry a bound (L_next is left alone)
  uint32_t workers;       // CTAs of finalize that process the candidates
  uint32_t seq;           // launch sequence number (tags the decision word)
};

__device__ __forceinline__ uint32_t key_of(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }
__device__ __forceinline__ uint32_t lanemask_lt() {
  uint32_t m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}
__device__ __forceinline__ uint32_t ld_volatile(const uint32_t* p) {
  return *reinterpret_cast<const volatile uint32_t*>(p);
}
__device__ __forceinline__ uint32_t part_first_tile(uint32_t part, uint32_t parts, uint32_t num_tiles) {
  return (uint32_t)((uint64_t)part * num_tiles / parts);
}

// ---- the value an element contributes to the selection ------------------------
// push (Algorithm 3):  t = fl(fl(m*u) + fl(eta*g));  Algorithm 1:  t = fl(u + fl(eta*g));  pull:  D.
template <int MODE>
__device__ __forceinline__ float combine(float u, float g, float m, float lr) {
  if (MODE == kPushSam) return __fadd_rn(__fmul_rn(m, u), __fmul_rn(lr, g));
  if (MODE == kPushResidual) return __fadd_rn(u, __fmul_rn(lr, g));
  return u;
}
// what a push stores for an element that is certainly not sent
template <int MODE>
__device__ __forceinline__ float unsent(float t, float inv_m) {
  return MODE == kPushSam ? __fmul_rn(t, inv_m) : t;
}

template <int MODE>
__device__ __forceinline__ void load_tile_vec(const float* __restrict__ a, const float* __restrict__ g,
                                              uint32_t start, int lane, float m, float lr,
                                              float (&x)[4 * kVecIters]) {
  const float4* pa = reinterpret_cast<const float4*>(a + start) + lane;
  float4 va[kVecIters];
#pragma unroll
  for (int j = 0; j < kVecIters; ++j) va[j] = __ldcs(pa + j * 32);
  if (MODE != kPull) {
    const float4* pg = reinterpret_cast<const float4*>(g + start) + lane;
    float4 vg[kVecIters];
#pragma unroll
    for (int j = 0; j < kVecIters; ++j) vg[j] = __ldcs(pg + j * 32);
#pragma unroll
    for (int j = 0; j < kVecIters; ++j) {
      x[4 * j + 0] = combine<MODE>(va[j].x, vg[j].x, m, lr);
      x[4 * j + 1] = combine<MODE>(va[j].y, vg[j].y, m, lr);
      x[4 * j + 2] = combine<MODE>(va[j].z, vg[j].z, m, lr);
      x[4 * j + 3] = combine<MODE>(va[j].w, vg[j].w, m, lr);
    }
  } else {
#pragma unroll
    for (int j = 0; j < kVecIters; ++j) {
      x[4 * j + 0] = va[j].x;
      x[4 * j + 1] = va[j].y;
      x[4 * j + 2] = va[j].z;
      x[4 * j + 3] = va[j].w;
    }
  }
}

// ---- stream pass ----------------------------------------------------------------
struct StreamShared {
  uint32_t hist[kBins1];  // top 11 key bits of the candidates of the layer being processed
  uint32_t cursor;        // candidates appended by this CTA so far
};

__device__ __forceinline__ void flush_hist(uint32_t* s_hist, uint32_t* g_hist) {
  for (int b = threadIdx.x; b < kBins1; b += kThreads) {
    const uint32_t v = s_hist[b];
    if (v) {
      atomicAdd(g_hist + b, v);
      s_hist[b] = 0;
    }
  }
}

// CTA `cta` of `G` handles a contiguous range of tiles, one tile per warp at a time,
// layer by layer, so that the CTA's shared histogram always belongs to one layer; it
// is added to the global one when the CTA leaves the layer.
template <int MODE>
__device__ void stream_tiles(const Workspace& ws, const SelArgs& a, const uint32_t* Larr,
                             const float* __restrict__ in, float* __restrict__ out, uint32_t cta, uint32_t G,
                             StreamShared& sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t t0 = part_first_tile(cta, G, ws.num_tiles), t1 = part_first_tile(cta + 1, G, ws.num_tiles);
  const uint32_t lt = lanemask_lt();
  for (int b = threadIdx.x; b < kBins1; b += kThreads) sh.hist[b] = 0;
  if (threadIdx.x == 0) {
    sh.cursor = 0;
    if (cta == 0) ws.sync[kParts] = G;
  }
  __syncthreads();
  if (t0 >= t1) {
    if (threadIdx.x == 0) {
      ws.part_cands[cta] = 0;
      ws.part_slot0[cta] = 0;
    }
    return;
  }
  const uint32_t slot0 = ws.tiles[t0].start;  // first slot of this CTA's region
  const uint32_t seg_first = ws.tiles[t0].seg, seg_last = ws.tiles[t1 - 1].seg;
  for (uint32_t s = seg_first; s <= seg_last; ++s) {
    const uint32_t a0 = max(t0, ws.segs[s].tile_begin), a1 = min(t1, ws.segs[s].tile_end);
    const uint32_t L = Larr[s];
    uint32_t t = a0 + warp;
    Tile next;
    next.start = 0; next.len = 0; next.seg = 0;
    if (t < a1) next = ws.tiles[t];
    for (; t < a1; t += kWarps) {
      const Tile tile = next;
      if (t + kWarps < a1) next = ws.tiles[t + kWarps];
      if (tile.len == kWarpTile) {
        float x[4 * kVecIters];
        load_tile_vec<MODE>(in, a.grad, tile.start, lane, a.m, a.lr, x);
        uint32_t mask = 0;
#pragma unroll
        for (int e = 0; e < 4 * kVecIters; ++e)
          if (key_of(x[e]) >= L) mask |= 1u << e;
        if (MODE != kPull) {
          float4* po = reinterpret_cast<float4*>(out + tile.start) + lane;
#pragma unroll
          for (int j = 0; j < kVecIters; ++j) {
            float4 o;
            o.x = (mask >> (j * 4 + 0)) & 1 ? x[4 * j + 0] : unsent<MODE>(x[4 * j + 0], a.inv_m);
            o.y = (mask >> (j * 4 + 1)) & 1 ? x[4 * j + 1] : unsent<MODE>(x[4 * j + 1], a.inv_m);
            o.z = (mask >> (j * 4 + 2)) & 1 ? x[4 * j + 2] : unsent<MODE>(x[4 * j + 2], a.inv_m);
            o.w = (mask >> (j * 4 + 3)) & 1 ? x[4 * j + 3] : unsent<MODE>(x[4 * j + 3], a.inv_m);
            __stcs(po + j * 32, o);
          }
        }
        const uint32_t total = __reduce_add_sync(kFull, (uint32_t)__popc(mask));
        if (total) {
          uint32_t base = 0;
          if (lane == 0) base = slot0 + atomicAdd(&sh.cursor, total);
          base = __shfl_sync(kFull, base, 0);
#pragma unroll
          for (int j = 0; j < kVecIters; ++j) {
            const uint32_t mj = (mask >> (j * 4)) & 0xFu;
            if (!__any_sync(kFull, mj != 0)) continue;
            const uint32_t b0 = __ballot_sync(kFull, mj & 1u), b1 = __ballot_sync(kFull, mj & 2u);
            const uint32_t b2 = __ballot_sync(kFull, mj & 4u), b3 = __ballot_sync(kFull, mj & 8u);
            uint32_t pos = base + __popc(b0 & lt) + __popc(b1 & lt) + __popc(b2 & lt) + __popc(b3 & lt);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              if ((mj >> c) & 1u) {
                const float v = x[4 * j + c];
                ws.cand_idx[pos] = tile.start + j * 128 + lane * 4 + c;
                ws.cand_val[pos] = v;
                atomicAdd(sh.hist + (key_of(v) >> 20), 1u);
                ++pos;
              }
            }
            base += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
          }
        }
      } else {
        // ragged tile (first or last of a layer): one element per lane and step.  The tile
        // has at most kWarpTile elements = 16 steps; candidate flags are kept as one bit per step.
        uint32_t flags = 0;
        for (int st = 0; st * 32 < (int)tile.len; ++st) {
          const uint32_t off = st * 32 + lane;
          if (off < tile.len) {
            const uint32_t i = tile.start + off;
            const float x = combine<MODE>(in[i], MODE != kPull ? a.grad[i] : 0.f, a.m, a.lr);
            const bool cand = key_of(x) >= L;
            if (MODE != kPull) out[i] = cand ? x : unsent<MODE>(x, a.inv_m);
            if (cand) flags |= 1u << st;
          }
        }
        const uint32_t total = __reduce_add_sync(kFull, (uint32_t)__popc(flags));
        if (total) {
          uint32_t base = 0;
          if (lane == 0) base = slot0 + atomicAdd(&sh.cursor, total);
          base = __shfl_sync(kFull, base, 0);
          for (int st = 0; st * 32 < (int)tile.len; ++st) {
            const bool cand = (flags >> st) & 1u;
            const uint32_t b = __ballot_sync(kFull, cand);
            if (cand) {
              // a candidate's value is what this thread just stored (push) or the input itself (pull)
              const uint32_t i = tile.start + st * 32 + lane;
              const float x = MODE == kPull ? in[i] : out[i];
              const uint32_t pos = base + __popc(b & lt);
              ws.cand_idx[pos] = i;
              ws.cand_val[pos] = x;
              atomicAdd(sh.hist + (key_of(x) >> 20), 1u);
            }
            base += __popc(b);
          }
        }
      }
    }
    __syncthreads();
    flush_hist(sh.hist, ws.hist1 + (size_t)s * kBins1);
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    ws.part_cands[cta] = sh.cursor;
    ws.part_slot0[cta] = slot0;
  }
}

// ---- histogram of ALL elements (top 11 key bits), for the bound that cannot fail ----
// Adds one warp-wide batch of bins to the shared histogram.  Lanes holding the same
// bin as lane 0's are counted with one ballot (values cluster in few bins: zeros in a
// sparse difference vector, the bulk of a bell-shaped gradient); the rest use atomics.
__device__ __forceinline__ void hist_add(uint32_t* s_hist, uint32_t bin, bool valid, int lane) {
  const uint32_t lead = __shfl_sync(kFull, bin, 0);
  const bool same = valid && bin == lead;
  const uint32_t b = __ballot_sync(kFull, same);
  if (lane == 0 && b) atomicAdd(s_hist + lead, (uint32_t)__popc(b));
  if (valid && !same) atomicAdd(s_hist + bin, 1u);
}

template <int MODE>
__device__ void hist_all_tiles(const Workspace& ws, const SelArgs& a, const float* __restrict__ in,
                               uint32_t cta, uint32_t G, uint32_t* s_hist) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t t0 = part_first_tile(cta, G, ws.num_tiles), t1 = part_first_tile(cta + 1, G, ws.num_tiles);
  for (int b = threadIdx.x; b < kBins1; b += kThreads) s_hist[b] = 0;
  __syncthreads();
  if (t0 >= t1) return;
  const uint32_t seg_first = ws.tiles[t0].seg, seg_last = ws.tiles[t1 - 1].seg;
  for (uint32_t s = seg_first; s <= seg_last; ++s) {
    const uint32_t a0 = max(t0, ws.segs[s].tile_begin), a1 = min(t1, ws.segs[s].tile_end);
    for (uint32_t t = a0 + warp; t < a1; t += kWarps) {
      const Tile tile = ws.tiles[t];
      if (tile.len == kWarpTile) {
        float x[4 * kVecIters];
        load_tile_vec<MODE>(in, a.grad, tile.start, lane, a.m, a.lr, x);
#pragma unroll
        for (int e = 0; e < 4 * kVecIters; ++e) hist_add(s_hist, key_of(x[e]) >> 20, true, lane);
      } else {
        for (uint32_t base = 0; base < tile.len; base += 32) {
          const uint32_t off = base + lane;
          const bool valid = off < tile.len;
          float x = 0.f;
          if (valid) {
            const uint32_t i = tile.start + off;
            x = combine<MODE>(in[i], MODE != kPull ? a.grad[i] : 0.f, a.m, a.lr);
          }
          hist_add(s_hist, key_of(x) >> 20, valid, lane);
        }
      }
    }
    __syncthreads();
    flush_hist(s_hist, ws.hist1 + (size_t)s * kBins1);
    __syncthreads();
  }
}

// ---- block-wide helpers (kThreads threads) -----------------------------------------
// exclusive scan of one 64-bit value per thread; `total` is the block sum
__device__ __forceinline__ unsigned long long block_excl_scan(unsigned long long v, unsigned long long* s_warp,
                                                              unsigned long long& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const unsigned long long o = __shfl_up_sync(kFull, inc, d);
    if (lane >= d) inc += o;
  }
  __syncthreads();  // s_warp may still be read from a previous call
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  unsigned long long base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) {
    const unsigned long long x = s_warp[w];
    if (w < warp) base += x;
    tot += x;
  }
  total = tot;
  return base + inc - v;
}

// From a histogram of B bins finds, counting from the top bin down, the bin that
// holds the k-th entry.  Returns total count; bin/krem are valid when total >= k:
// krem = k minus the entries in bins above `bin` (1 <= krem <= hist[bin]).
template <int B>
__device__ uint32_t block_pick(const uint32_t* hist, uint32_t k, uint32_t& bin, uint32_t& krem,
                               unsigned long long* s_warp, uint32_t* s_res) {
  constexpr int PER = B / kThreads;
  uint32_t loc[PER];
  uint32_t sum = 0;
  // thread 0 owns the top PER bins, thread 1 the next PER, ...
  const int top = B - 1 - threadIdx.x * PER;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    loc[j] = __ldcg(hist + top - j);
    sum += loc[j];
  }
  unsigned long long total;
  const uint32_t above = (uint32_t)block_excl_scan(sum, s_warp, total);
  if (above < k && k <= above + sum) {
    uint32_t acc = above;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (acc < k && k <= acc + loc[j]) {
        s_res[0] = (uint32_t)(top - j);
        s_res[1] = k - acc;
      }
      acc += loc[j];
    }
  }
  __syncthreads();
  bin = s_res[0];
  krem = s_res[1];
  __syncthreads();
  return (uint32_t)total;
}

// Barrier among the first W CTAs of the grid (all resident: cooperative launch).
// Bounded: returns false, with the status word set, if the others do not arrive.
__device__ bool worker_barrier(uint32_t* sync, uint32_t W, int* status, int* s_ok) {
  __syncthreads();
  if (threadIdx.x == 0) {
    int ok = 1;
    __threadfence();
    const uint32_t gen = ld_volatile(sync + kBarGen);
    const uint32_t prev = atomicAdd(sync + kBarCount, 1u);
    if (prev == W - 1) {
      atomicExch(sync + kBarCount, 0u);
      __threadfence();
      atomicAdd(sync + kBarGen, 1u);
    } else {
      uint32_t spins = 0;
      while (ld_volatile(sync + kBarGen) == gen) {
        if (++spins > kSpinLimit) {
          ok = 0;
          atomicMin(status, kStatusTimeout);
          break;
        }
        __nanosleep(20);
      }
    }
    __threadfence();
    *s_ok = ok;
  }
  __syncthreads();
  return *s_ok != 0;
}

// ---- finalize -------------------------------------------------------------------
// The candidates are numbered flat over the parts: part p holds part_cands[p] of them in
// consecutive slots from part_slot0[p] on, tile after tile (the tiles of a part in the
// order its warps happened to finish them, each tile's candidates in index order).
// Every phase below is one flat loop over that numbering; the layer and the tile of a
// candidate follow from its index.
constexpr int kSegCap = 1024;  // layers whose tables fit in shared memory; more fall back to global reads

struct FinalizeShared {
  StreamShared stream;                 // only used when the guess failed and the passes are redone here
  unsigned long long warp_scan[kWarps];
  uint32_t res[2];
  int ok;
  uint32_t pre_cands[kMaxGrid + 1];    // exclusive prefix of part_cands
  uint32_t slot0[kMaxGrid];            // first slot of each part
  uint2 base[kMaxWorkers];             // exclusive prefix of the scanning CTAs' (gt, eq) totals
  uint32_t seg_off[kSegCap + 1];       // first element of each layer, and n
  uint32_t seg_tile0[kSegCap];         // first tile of each layer
  uint32_t seg_a[kSegCap];             // per-layer parameter of the current phase (prefix, or T)
  uint32_t seg_b[kSegCap];             // second one (r)
  uint2 seg_start[kSegCap];            // (gt, eq) counted before the layer's first tile
};

struct SegView {  // per-layer tables, in shared memory when they fit
  const uint32_t* off;
  const uint32_t* tile0;
  uint32_t S;
};

// layer that holds element i: last s with off[s] <= i
__device__ __forceinline__ uint32_t seg_of(const SegView& v, uint32_t i) {
  uint32_t lo = 0, hi = v.S - 1;
  while (lo < hi) {
    const uint32_t mid = (lo + hi + 1) >> 1;
    if (v.off[mid] <= i) lo = mid; else hi = mid - 1;
  }
  return lo;
}
// tiles of a layer are cut at the multiples of kWarpTile of the global index
__device__ __forceinline__ uint32_t tile_of(const SegView& v, uint32_t seg, uint32_t i) {
  return v.tile0[seg] + (i / kWarpTile - v.off[seg] / kWarpTile);
}
// slot of flat candidate p: last part with pre[part] <= p
__device__ __forceinline__ uint32_t slot_of(const FinalizeShared& sh, uint32_t parts, uint32_t p, uint32_t* part_out) {
  uint32_t lo = 0, hi = parts - 1;
  while (lo < hi) {
    const uint32_t mid = (lo + hi + 1) >> 1;
    if (sh.pre_cands[mid] <= p) lo = mid; else hi = mid - 1;
  }
  if (part_out) *part_out = lo;
  return sh.slot0[lo] + (p - sh.pre_cands[lo]);
}

template <int MODE>
__global__ void __launch_bounds__(kThreads, 2) k_finalize(Workspace ws, SelArgs a) {
  __shared__ FinalizeShared sh;

  constexpr int PM = MODE == kPull ? 1 : 0;
  const uint32_t cta = blockIdx.x, W = gridDim.x, S = ws.num_segs;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t lt = lanemask_lt();
  const uint32_t gthread = cta * kThreads + threadIdx.x, nthreads = W * kThreads;

  // pointers are read once, before anything may exchange them
  const float* in = nullptr;
  float* out = nullptr;
  if (MODE == kPull) {
    in = a.D;
  } else {
    in = *a.u_cur_slot;
    out = *a.u_spare_slot;
  }

  // layer tables
  const bool seg_smem = S <= (uint32_t)kSegCap;
  if (seg_smem) {
    for (uint32_t s = threadIdx.x; s <= S; s += kThreads) sh.seg_off[s] = ws.seg_off[s];
    for (uint32_t s = threadIdx.x; s < S; s += kThreads) sh.seg_tile0[s] = ws.segs[s].tile_begin;
  }
  SegView sv;
  sv.off = seg_smem ? sh.seg_off : ws.seg_off;
  sv.tile0 = seg_smem ? sh.seg_tile0 : ws.seg_tile0;
  sv.S = S;
  __syncthreads();

  bool redo = false;
  for (int attempt = 0; attempt < 2; ++attempt) {
    if (redo) {
      // the guess was too high for some layer: take the bound that cannot fail from a histogram of
      // the whole input and repeat the stream pass, with the few CTAs this kernel has
      hist_all_tiles<MODE>(ws, a, in, cta, W, sh.stream.hist);
      if (!worker_barrier(ws.sync, W, ws.status, &sh.ok)) return;
      for (uint32_t s = cta; s < S; s += W) {
        uint32_t bin, krem;
        uint32_t* h = ws.hist1 + (size_t)s * kBins1;
        block_pick<kBins1>(h, ws.segs[s].k[PM], bin, krem, sh.warp_scan, sh.res);
        if (threadIdx.x == 0) ws.L_safe[s] = bin << 20;
        for (int b = threadIdx.x; b < kBins1; b += kThreads) h[b] = 0;
      }
      if (cta == 0 && threadIdx.x == 0) ws.sync[kFail] = 0;
      if (!worker_barrier(ws.sync, W, ws.status, &sh.ok)) return;
      stream_tiles<MODE>(ws, a, ws.L_safe, in, out, cta, W, sh.stream);
      if (!worker_barrier(ws.sync, W, ws.status, &sh.ok)) return;
    }
    // level 1: pick the bin of the k-th largest among the candidates; check the guess
    for (uint32_t s = cta; s < S; s += W) {
      uint32_t bin, krem;
      uint32_t* h = ws.hist1 + (size_t)s * kBins1;
      const uint32_t k = ws.segs[s].k[PM];
      const uint32_t total = block_pick<kBins1>(h, k, bin, krem, sh.warp_scan, sh.res);
      if (total < k) {
        if (threadIdx.x == 0) atomicOr(ws.sync + kFail, 1u);
      } else {
        if (threadIdx.x == 0) {
          ws.sel[s].prefix = bin;
          ws.sel[s].krem = krem;
          atomicAdd(ws.stats + 2, (unsigned long long)total);
        }
        if (a.speculate) {
          // bound suggested for a later selection on this layer
          const uint32_t want = max(k * kSpecFactor, k + kSpecSlack);
          uint32_t lbin, lrem;
          if (total >= want) {
            block_pick<kBins1>(h, want, lbin, lrem, sh.warp_scan, sh.res);
          } else {
            const uint32_t used = (redo ? __ldcg(ws.L_safe + s) : a.L_in[s]) >> 20;
            lbin = used > 0 ? used - 1 : 0;
          }
          __syncthreads();
          if (threadIdx.x == 0) a.L_next[s] = lbin << 20;
        }
      }
      __syncthreads();
      for (int b = threadIdx.x; b < kBins1; b += kThreads) h[b] = 0;
    }
    if (!worker_barrier(ws.sync, W, ws.status, &sh.ok)) return;
    if (redo || ld_volatile(ws.sync + kFail) == 0) break;
    redo = true;
  }

  // flat numbering of the candidates
  const uint32_t parts = ld_volatile(ws.sync + kParts);
  {
    unsigned long long carry = 0;
    for (uint32_t base = 0; base < parts; base += kThreads) {
      const uint32_t p = base + threadIdx.x;
      const unsigned long long v = p < parts ? __ldcg(ws.part_cands + p) : 0;
      unsigned long long total;
      const unsigned long long ex = block_excl_scan(v, sh.warp_scan, total) + carry;
      if (p < parts) {
        sh.pre_cands[p] = (uint32_t)ex;
        sh.slot0[p] = __ldcg(ws.part_slot0 + p);
      }
      carry += total;
    }
    if (threadIdx.x == 0) sh.pre_cands[parts] = (uint32_t)carry;
    __syncthreads();
  }
  const uint32_t C = sh.pre_cands[parts];

  // ---- levels 2 and 3 ----------------------------------------------------------------
#pragma unroll 1
  for (int level = 2; level <= 3; ++level) {
    uint32_t* hist = level == 2 ? ws.hist2 : ws.hist3;
    const int B = level == 2 ? kBins2 : kBins3;   // both 1024
    const int SH = level == 2 ? 20 : 10;
    if (seg_smem) {
      for (uint32_t s = threadIdx.x; s < S; s += kThreads) sh.seg_a[s] = __ldcg(&ws.sel[s].prefix);
      __syncthreads();
    }
    for (uint32_t p = gthread; p < C; p += nthreads) {
      const uint32_t slot = slot_of(sh, parts, p, nullptr);
      const uint32_t key = key_of(__ldcg(ws.cand_val + slot));
      uint32_t seg = 0;
      if (S > 1) seg = seg_of(sv, __ldcg(ws.cand_idx + slot));
      const uint32_t prefix = seg_smem ? sh.seg_a[seg] : __ldcg(&ws.sel[seg].prefix);
      if ((key >> SH) == prefix) atomicAdd(hist + (size_t)seg * B + ((key >> (SH - 10)) & 1023u), 1u);
    }
    if (!worker_barrier(ws.sync, W, ws.status, &sh.ok)) return;
    for (uint32_t s = cta; s < S; s += W) {
      uint32_t bin, krem;
      uint32_t* h = hist + (size_t)s * B;
      block_pick<kBins2>(h, __ldcg(&ws.sel[s].krem), bin, krem, sh.warp_scan, sh.res);
      if (threadIdx.x == 0) {
        const uint32_t pre = (__ldcg(&ws.sel[s].prefix) << 10) | bin;
        ws.sel[s].prefix = pre;
        ws.sel[s].krem = krem;
        if (level == 3) {
          ws.sel[s].T = pre;   // all 31 key bits are fixed now
          ws.sel[s].r = krem;
        }
      }
      for (int b = threadIdx.x; b < B; b += kThreads) h[b] = 0;
    }
    if (!worker_barrier(ws.sync, W, ws.status, &sh.ok)) return;
  }

  // ---- count: per tile, how many candidates have key > T and key == T ----------------
  // (tile_sel is all zero on entry: the scan below clears what it reads)
  if (seg_smem) {
    for (uint32_t s = threadIdx.x; s < S; s += kThreads) {
      sh.seg_a[s] = __ldcg(&ws.sel[s].T);
      sh.seg_b[s] = __ldcg(&ws.sel[s].r);
    }
    __syncthreads();
  }
  for (uint32_t p = gthread; p < C; p += nthreads) {
    const uint32_t slot = slot_of(sh, parts, p, nullptr);
    const uint32_t key = key_of(__ldcg(ws.cand_val + slot));
    const uint32_t idx = __ldcg(ws.cand_idx + slot);
    const uint32_t seg = S > 1 ? seg_of(sv, idx) : 0;
    const uint32_t T = seg_smem ? sh.seg_a[seg] : __ldcg(&ws.sel[seg].T);
    if (key >= T) {
      uint2* c = ws.tile_sel + tile_of(sv, seg, idx);
      atomicAdd(key > T ? &c->x : &c->y, 1u);
    }
  }
  if (!worker_barrier(ws.sync, W, ws.status, &sh.ok)) return;

  // ---- scan over the tiles in index order: CTA c owns tiles [c*chunk, (c+1)*chunk) ----
  const uint32_t chunk_tiles = (ws.num_tiles + W - 1) / W;
  {
    const uint32_t t0 = min(ws.num_tiles, cta * chunk_tiles), t1 = min(ws.num_tiles, t0 + chunk_tiles);
    unsigned long long carry = 0;
    for (uint32_t base = t0; base < t1; base += kThreads) {
      const uint32_t t = base + threadIdx.x;
      unsigned long long v = 0;
      if (t < t1) {
        const uint2 c = __ldcg(ws.tile_sel + t);
        v = ((unsigned long long)c.x << 32) | c.y;
        if (v) ws.tile_sel[t] = make_uint2(0, 0);
      }
      unsigned long long total;
      const unsigned long long ex = block_excl_scan(v, sh.warp_scan, total) + carry;
      if (t < t1) ws.tile_pre[t] = make_uint2((uint32_t)(ex >> 32), (uint32_t)ex);
      carry += total;
    }
    if (threadIdx.x == 0) ws.cta_tot[cta] = make_uint2((uint32_t)(carry >> 32), (uint32_t)carry);
  }
  if (!worker_barrier(ws.sync, W, ws.status, &sh.ok)) return;

  // ---- emit: packet in index order, and the state updates that depend on selection ----
  {
    unsigned long long carry = 0;  // exclusive prefix of the CTAs' totals (W <= kMaxWorkers)
    for (uint32_t base = 0; base < W; base += kThreads) {
      const uint32_t c = base + threadIdx.x;
      unsigned long long v = 0;
      if (c < W) {
        const uint2 q = __ldcg(ws.cta_tot + c);
        v = ((unsigned long long)q.x << 32) | q.y;
      }
      unsigned long long total;
      const unsigned long long ex = block_excl_scan(v, sh.warp_scan, total) + carry;
      if (c < W) sh.base[c] = make_uint2((uint32_t)(ex >> 32), (uint32_t)ex);
      carry += total;
    }
    __syncthreads();
    // (gt, eq) counted before tile t, over all layers
    auto before_tile = [&](uint32_t t) {
      const uint2 pre = __ldcg(ws.tile_pre + t), b = sh.base[t / chunk_tiles];
      return make_uint2(b.x + pre.x, b.y + pre.y);
    };
    if (seg_smem) {
      for (uint32_t s = threadIdx.x; s < S; s += kThreads) sh.seg_start[s] = before_tile(sh.seg_tile0[s]);
      __syncthreads();
    }
    const uint32_t gwarp = cta * kWarps + warp, nwarps = W * kWarps;
    for (uint32_t c0 = gwarp * 32; c0 < C; c0 += nwarps * 32) {
      const uint32_t p = c0 + lane;
      const bool valid = p < C;
      uint32_t part = 0, idx = 0, key = 0, seg = 0, tile = 0xFFFFFFFFu, T = 0, r = 0;
      float val = 0.f;
      if (valid) {
        const uint32_t slot = slot_of(sh, parts, p, &part);
        idx = __ldcg(ws.cand_idx + slot);
        val = __ldcg(ws.cand_val + slot);
        key = key_of(val);
        seg = S > 1 ? seg_of(sv, idx) : 0;
        tile = tile_of(sv, seg, idx);
        T = seg_smem ? sh.seg_a[seg] : __ldcg(&ws.sel[seg].T);
        r = seg_smem ? sh.seg_b[seg] : __ldcg(&ws.sel[seg].r);
      }
      const bool is_gt = valid && key > T, is_eq = valid && key == T;
      const uint32_t bgt = __ballot_sync(kFull, is_gt), beq = __ballot_sync(kFull, is_eq);
      // the candidates of one tile are consecutive: a lane starts a tile if its left neighbour is in another one
      const uint32_t left = __shfl_up_sync(kFull, tile, 1);
      const uint32_t heads = __ballot_sync(kFull, lane == 0 || left != tile);
      const int head = 31 - __clz(heads & (lt | (1u << lane)));       // first lane of my tile in this step
      const uint32_t mine = lt & ~((1u << head) - 1u);                  // lanes of my tile before me
      // the tile of lane 0 may have started in earlier slots of the same part: count what it holds there
      uint32_t carry_gt = 0, carry_eq = 0;
      {
        const uint32_t tile0 = __shfl_sync(kFull, tile, 0), part0 = __shfl_sync(kFull, part, 0);
        const uint32_t T0 = __shfl_sync(kFull, T, 0), seg0 = __shfl_sync(kFull, seg, 0);
        const uint32_t first = sh.pre_cands[part0];                     // flat number of the part's first candidate
        uint32_t back = c0;
        while (back > first) {                                          // warp-uniform
          const uint32_t lo = back - min(back - first, 32u);
          const uint32_t pp = lo + lane;
          bool same = false;
          uint32_t k2 = 0;
          if (pp < back) {
            const uint32_t slot = sh.slot0[part0] + (pp - first);
            const uint32_t i2 = __ldcg(ws.cand_idx + slot);
            const uint32_t s2 = S > 1 ? seg_of(sv, i2) : 0;
            same = s2 == seg0 && tile_of(sv, s2, i2) == tile0;
            k2 = key_of(__ldcg(ws.cand_val + slot));
          }
          const uint32_t bs = __ballot_sync(kFull, same);
          carry_gt += __popc(__ballot_sync(kFull, same && k2 > T0));
          carry_eq += __popc(__ballot_sync(kFull, same && k2 == T0));
          if (bs != __ballot_sync(kFull, pp < back)) break;             // reached another tile
          back = lo;
        }
      }
      if (valid) {
        const uint2 tb = before_tile(tile);
        const uint2 s0 = seg_smem ? sh.seg_start[seg] : before_tile(sv.tile0[seg]);
        uint32_t gt_before = (tb.x - s0.x) + __popc(bgt & mine);
        uint32_t eq_before = (tb.y - s0.y) + __popc(beq & mine);
        if (head == 0) {
          gt_before += carry_gt;
          eq_before += carry_eq;
        }
        const bool sel = is_gt || (is_eq && eq_before < r);
        if (sel) {
          const uint32_t pos = ws.segs[seg].pkt_off[PM] + gt_before + min(eq_before, r);
          if (pos < a.pkt_count) {
            a.pkt_idx[pos] = idx;
            a.pkt_val[pos] = val;
          } else {
            atomicMin(ws.status, -1000 - MODE);
          }
          if (MODE == kPushResidual) out[idx] = 0.f;       // Algorithm 1: the sent part leaves v
          if (MODE == kPull) {
            a.D[idx] = 0.f;                                // Eq. 6b: v_k <- v_k + G
            if (a.theta_local) a.theta_local[idx] = __fadd_rn(a.theta_local[idx], val);  // Eq. 5
          }
        } else {
          if (MODE == kPushSam) out[idx] = __fmul_rn(val, a.inv_m);  // Eq. 12, lower branch
        }
      }
    }
  }
  if (cta == 0 && threadIdx.x == 0) {
    if (MODE != kPull) {  // the spare buffer now holds the worker's velocity
      float* cur = *a.u_cur_slot;
      *a.u_cur_slot = *a.u_spare_slot;
      *a.u_spare_slot = cur;
    }
    atomicAdd(ws.stats + ((redo || a.force_two_pass) ? 1 : 0), 1ull);
  }
}

// ---- the two passes as kernels of their own, for a selection with nothing to go by -------
template <int MODE>
__global__ void __launch_bounds__(kThreads, 4) k_hist_all(Workspace ws, SelArgs a) {
  __shared__ uint32_t s_hist[kBins1];
  const float* in = MODE == kPull ? a.D : *a.u_cur_slot;
  hist_all_tiles<MODE>(ws, a, in, blockIdx.x, gridDim.x, s_hist);
}

// one CTA per layer (strided): L_safe = lower edge of the top-11-bit bin holding the k-th largest key
template <int MODE>
__global__ void __launch_bounds__(kThreads) k_pick_lower(Workspace ws) {
  __shared__ unsigned long long s_warp[kWarps];
  __shared__ uint32_t s_res[2];
  constexpr int PM = MODE == kPull ? 1 : 0;
  for (uint32_t s = blockIdx.x; s < ws.num_segs; s += gridDim.x) {
    uint32_t bin, krem;
    uint32_t* h = ws.hist1 + (size_t)s * kBins1;
    block_pick<kBins1>(h, ws.segs[s].k[PM], bin, krem, s_warp, s_res);
    if (threadIdx.x == 0) ws.L_safe[s] = bin << 20;
    for (int b = threadIdx.x; b < kBins1; b += kThreads) h[b] = 0;
  }
}

// ---- stand-alone stream pass with the carried bound -------------------------------
template <int MODE>
__global__ void __launch_bounds__(kThreads, 4) k_stream(Workspace ws, SelArgs a) {
  __shared__ StreamShared sh;
  const float* in;
  float* out = nullptr;
  if (MODE == kPull) {
    in = a.D;
  } else {
    in = *a.u_cur_slot;
    out = *a.u_spare_slot;
  }
  stream_tiles<MODE>(ws, a, a.L_in, in, out, blockIdx.x, gridDim.x, sh);
}

// ---- server apply ---------------------------------------------------------------
// buffer q < N is D_q, buffer N is theta.  Indices of one packet are distinct, so every
// (buffer, entry) pair is touched by exactly one thread: plain load / subtract / store.
__global__ void __launch_bounds__(kThreads) k_scatter_sub(const uint32_t* __restrict__ idx,
                                                          const float* __restrict__ val, uint32_t count,
                                                          float* __restrict__ theta, float* __restrict__ D,
                                                          uint64_t d_stride, uint32_t num_workers, uint64_t n,
                                                          int* status) {
  const uint32_t j = blockIdx.x * kThreads + threadIdx.x;
  if (j >= count) return;
  const uint32_t i = idx[j];
  const float v = val[j];
  if (i >= n) {
    atomicMin(status, -2000);
    return;
  }
  const uint32_t q = blockIdx.y;
  float* p = (q == num_workers ? theta : D + (uint64_t)q * d_stride) + i;
  *p = __fsub_rn(*p, v);
}

}  // namespace dgs
