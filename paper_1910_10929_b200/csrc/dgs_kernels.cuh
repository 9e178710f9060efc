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
constexpr uint32_t kSpecFactor = 2; // aim for max(2k, k+64) candidates next time
constexpr uint32_t kSpecSlack = 64;
constexpr int kMaxGrid = 1024;      // upper bound on the grid of a stream pass (= parts of the candidate buffer)
constexpr int kMaxWorkers = 320;    // upper bound on the grid of finalize
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
  uint32_t* L_wide;       // [S] from the same histogram: the bound that admits max(3k, k+64) entries
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
  uint32_t* blk_max;      // pull: per block of kWarpTile elements, an upper bound on the keys of D_w in it (or null)
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
constexpr int kLiveWords = 128;     // one bit per stage-sized chunk of a CTA's share of a layer
struct StreamShared {
  uint32_t hist[kBins1];  // top 11 key bits of the candidates of the layer being processed
  uint32_t cursor;        // candidates appended by this CTA so far
  uint32_t live[kLiveWords];  // pull: chunks that may hold a candidate (the others are not read)
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

// What follows the loads of a full tile: x[16] holds this lane's values (4 float4 at
// elements j*128 + lane*4 + c of the tile).  Writes the new velocity (push), appends the
// tile's candidates in index order to the CTA's region, histograms their top key bits.
template <int MODE>
__device__ __forceinline__ void finish_full_tile(const Workspace& ws, const SelArgs& a, StreamShared& sh,
                                                 uint32_t tile_start, const float (&x)[4 * kVecIters], uint32_t L,
                                                 uint32_t slot0, int lane, uint32_t lt, float* __restrict__ out) {
  uint32_t mask = 0;
#pragma unroll
  for (int e = 0; e < 4 * kVecIters; ++e)
    if (key_of(x[e]) >= L) mask |= 1u << e;
  if (MODE != kPull) {
    float4* po = reinterpret_cast<float4*>(out + tile_start) + lane;
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
          ws.cand_idx[pos] = tile_start + j * 128 + lane * 4 + c;
          ws.cand_val[pos] = v;
          atomicAdd(sh.hist + (key_of(v) >> 20), 1u);
          ++pos;
        }
      }
      base += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
    }
  }
}

// A ragged tile (first or last of a layer, fewer than kWarpTile elements or not 16-byte
// aligned): one element per lane and step, straight from global memory.  At most 16
// steps; candidate flags are kept as one bit per step.
template <int MODE>
__device__ __forceinline__ void ragged_tile(const Workspace& ws, const SelArgs& a, StreamShared& sh, const Tile tile,
                                            uint32_t L, uint32_t slot0, int lane, uint32_t lt,
                                            const float* __restrict__ in, float* __restrict__ out) {
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

// CTA `cta` of `G` handles a contiguous range of tiles, one tile per warp at a time,
// layer by layer, so that the CTA's shared histogram always belongs to one layer; it
// is added to the global one when the CTA leaves the layer.  Loads go straight from
// global memory to registers (used where only a few CTAs run the pass).
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
        finish_full_tile<MODE>(ws, a, sh, tile.start, x, L, slot0, lane, lt, out);
      } else {
        ragged_tile<MODE>(ws, a, sh, tile, L, slot0, lane, lt, in, out);
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

// The same for a tile staged in shared memory (su: the tile of the state vector, sg: the
// tile of the gradient, push only).  The cost beyond the streaming part is kept
// proportional to the number of candidates: one packed warp scan gives every lane the
// rank of its candidates (lane l holds elements j*128 + l*4 + c, order is j-major, so the
// four per-j counts travel as four bytes of one word), and a lane that has candidates
// walks its set bits and recomputes their values from shared memory.
template <int MODE>
__device__ __forceinline__ void finish_full_tile_smem(const Workspace& ws, const SelArgs& a, StreamShared& sh,
                                                      uint32_t tile_start, const float* su, const float* sg,
                                                      uint32_t L, uint32_t slot0, int lane,
                                                      float* __restrict__ out) {
  const float Lf = __uint_as_float(L);   // |x| >= Lf  <=>  key(x) >= L for finite x (no flush-to-zero)
  const float4* pu = reinterpret_cast<const float4*>(su) + lane;
  const float4* pg = reinterpret_cast<const float4*>(sg) + lane;
  uint32_t mask = 0;
  uint32_t top = 0;       // pull: largest key of this lane's elements
#pragma unroll
  for (int j = 0; j < kVecIters; ++j) {
    float4 x = pu[j * 32];
    if (MODE == kPull) top = max(max(top, max(key_of(x.x), key_of(x.y))), max(key_of(x.z), key_of(x.w)));
    if (MODE != kPull) {
      const float4 g = pg[j * 32];
      x.x = combine<MODE>(x.x, g.x, a.m, a.lr);
      x.y = combine<MODE>(x.y, g.y, a.m, a.lr);
      x.z = combine<MODE>(x.z, g.z, a.m, a.lr);
      x.w = combine<MODE>(x.w, g.w, a.m, a.lr);
    }
    const bool c0 = fabsf(x.x) >= Lf, c1 = fabsf(x.y) >= Lf, c2 = fabsf(x.z) >= Lf, c3 = fabsf(x.w) >= Lf;
    mask |= ((c0 ? 1u : 0u) | (c1 ? 2u : 0u) | (c2 ? 4u : 0u) | (c3 ? 8u : 0u)) << (4 * j);
    if (MODE != kPull) {
      float4 o;
      o.x = c0 ? x.x : unsent<MODE>(x.x, a.inv_m);
      o.y = c1 ? x.y : unsent<MODE>(x.y, a.inv_m);
      o.z = c2 ? x.z : unsent<MODE>(x.z, a.inv_m);
      o.w = c3 ? x.w : unsent<MODE>(x.w, a.inv_m);
      __stcs(reinterpret_cast<float4*>(out + tile_start) + lane + j * 32, o);
    }
  }
  if (MODE == kPull && a.blk_max != nullptr) {
    // the tile is a whole block: its bound becomes exact again (entries sent later only lower it)
    top = __reduce_max_sync(kFull, top);
    if (lane == 0) a.blk_max[tile_start / kWarpTile] = top;
  }
  if (!__any_sync(kFull, mask != 0)) return;
  // per-j candidate counts of this lane, one per byte
  uint32_t t = mask - ((mask >> 1) & 0x5555u);
  t = (t & 0x3333u) + ((t >> 2) & 0x3333u);                       // nibble j = count of nibble j of mask
  const uint32_t packed = (t & 0xFu) | ((t & 0xF0u) << 4) | ((t & 0xF00u) << 8) | ((t & 0xF000u) << 12);
  uint32_t incl = packed;                                          // byte j: inclusive prefix over lanes (<= 128)
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t o = __shfl_up_sync(kFull, incl, d);
    if (lane >= d) incl += o;
  }
  const uint32_t tot = __shfl_sync(kFull, incl, 31);
  const uint32_t t0 = tot & 0xFFu, t1 = (tot >> 8) & 0xFFu, t2 = (tot >> 16) & 0xFFu, t3 = tot >> 24;
  uint32_t base = 0;
  if (lane == 0) base = slot0 + atomicAdd(&sh.cursor, t0 + t1 + t2 + t3);
  base = __shfl_sync(kFull, base, 0);
  if (mask) {
    const uint32_t excl = incl - packed;                           // byte j: candidates of lower lanes at step j
    uint32_t m = mask;
    while (m) {
      const int e = __ffs(m) - 1;
      m &= m - 1;
      const int j = e >> 2, c = e & 3;
      const uint32_t before_j = j == 0 ? 0u : (j == 1 ? t0 : (j == 2 ? t0 + t1 : t0 + t1 + t2));
      const uint32_t in_lane = __popc((mask >> (4 * j)) & ((1u << c) - 1u));
      const uint32_t pos = base + before_j + ((excl >> (8 * j)) & 0xFFu) + in_lane;
      const uint32_t off = j * 128 + lane * 4 + c;
      const float v = combine<MODE>(su[off], MODE != kPull ? sg[off] : 0.f, a.m, a.lr);
      ws.cand_idx[pos] = tile_start + off;
      ws.cand_val[pos] = v;
      atomicAdd(sh.hist + (key_of(v) >> 20), 1u);
    }
  }
}

// ---- the same pass with TMA-staged tiles --------------------------------------------
// Full tiles are brought into a ring of shared-memory stages by bulk asynchronous copies
// (cp.async.bulk, completion counted on an mbarrier per stage), kStageTiles tiles of each
// input per stage, so that several stages are in flight while the warps work on one: the
// bytes in flight no longer depend on how many warps are waiting at a load.
constexpr int kStageTiles = kWarps;                        // one tile per warp and stage
constexpr int kStageFloats = kStageTiles * kWarpTile;      // per input array
template <int MODE> struct StreamRing {
  static constexpr int kInputs = MODE == kPull ? 1 : 2;
  static constexpr int kStages = MODE == kPull ? 3 : 2;
  static constexpr int kStageBytes = kInputs * kStageFloats * 4;
  static constexpr int kBytes = kStages * kStageBytes;     // 80 KB (pull) / 96 KB (push)
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// bounded wait: false if the copies did not land within the poll limit
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  for (uint32_t spins = 0; spins < kSpinLimit; ++spins)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// global -> shared bulk copy; src and dst 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

template <int MODE>
__device__ void stream_tiles_tma(const Workspace& ws, const SelArgs& a, const uint32_t* Larr,
                                 const float* __restrict__ in, float* __restrict__ out, uint32_t cta, uint32_t G,
                                 StreamShared& sh, float* ring, uint64_t* full, int* s_dead) {
  using R = StreamRing<MODE>;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t t0 = part_first_tile(cta, G, ws.num_tiles), t1 = part_first_tile(cta + 1, G, ws.num_tiles);
  const uint32_t lt = lanemask_lt();
  for (int b = threadIdx.x; b < kBins1; b += kThreads) sh.hist[b] = 0;
  if (threadIdx.x == 0) {
    sh.cursor = 0;
    *s_dead = 0;
    if (cta == 0) ws.sync[kParts] = G;
    for (int st = 0; st < R::kStages; ++st) mbar_init(full + st, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (t0 >= t1) {
    if (threadIdx.x == 0) {
      ws.part_cands[cta] = 0;
      ws.part_slot0[cta] = 0;
    }
    return;
  }
  const uint32_t slot0 = ws.tiles[t0].start;
  const uint32_t seg_first = ws.tiles[t0].seg, seg_last = ws.tiles[t1 - 1].seg;
  uint32_t uses = 0;  // stage uses so far (same in every thread): stage = use % kStages, parity = (use / kStages) & 1
  for (uint32_t s = seg_first; s <= seg_last; ++s) {
    const uint32_t a0 = max(t0, ws.segs[s].tile_begin), a1 = min(t1, ws.segs[s].tile_end);
    const uint32_t L = Larr[s];
    // only the first and the last tile of a layer can be ragged
    const bool head = ws.tiles[a0].len != kWarpTile;
    const bool tail = (a1 - 1 > a0 || !head) && ws.tiles[a1 - 1].len != kWarpTile;
    const uint32_t f0 = a0 + (head ? 1u : 0u), f1 = a1 - (tail ? 1u : 0u);   // full tiles [f0, f1)
    if (head && warp == 0) ragged_tile<MODE>(ws, a, sh, ws.tiles[a0], L, slot0, lane, lt, in, out);
    if (tail && warp == 1) ragged_tile<MODE>(ws, a, sh, ws.tiles[a1 - 1], L, slot0, lane, lt, in, out);
    const uint32_t nfull = f1 > f0 ? f1 - f0 : 0;
    const uint32_t nchunks = (nfull + kStageTiles - 1) / kStageTiles;
    const uint32_t e0 = nfull ? ws.tiles[f0].start : 0;   // first element of the full tiles (multiple of kWarpTile)
    auto issue = [&](uint32_t chunk, uint32_t use) {      // thread 0 only
      const uint32_t st = use % R::kStages;
      const uint32_t tiles_here = min((uint32_t)kStageTiles, nfull - chunk * kStageTiles);
      const uint32_t bytes = tiles_here * kWarpTile * 4;
      const size_t elem = (size_t)e0 + (size_t)chunk * kStageFloats;
      float* dst = ring + (size_t)st * (R::kStageBytes / 4);
      mbar_expect_tx(full + st, bytes * R::kInputs);
      bulk_load(dst, in + elem, bytes, full + st);
      if (MODE != kPull) bulk_load(dst + kStageFloats, a.grad + elem, bytes, full + st);
    };
    // Pull: a chunk all of whose blocks have a bound below L holds no candidate and is not read.
    const bool can_skip = MODE == kPull && a.blk_max != nullptr && L > 0 && nchunks <= kLiveWords * 32;
    if (can_skip) {
      for (uint32_t base = warp * 32; base < nchunks; base += kWarps * 32) {
        const uint32_t c = base + lane;
        bool live = false;
        if (c < nchunks) {
          const uint32_t tiles_here = min((uint32_t)kStageTiles, nfull - c * kStageTiles);
          const uint32_t* bm = a.blk_max + e0 / kWarpTile + c * kStageTiles;
          uint32_t top = 0;
          for (uint32_t j = 0; j < tiles_here; ++j) top = max(top, __ldcg(bm + j));
          live = top >= L;
        }
        const uint32_t word = __ballot_sync(kFull, live);
        if (lane == 0) sh.live[base / 32] = word;
      }
      __syncthreads();
    }
    auto next_live = [&](uint32_t c) -> uint32_t {       // first chunk >= c that is read, nchunks if none
      if constexpr (MODE == kPull) {
        while (can_skip && c < nchunks) {
          const uint32_t w = sh.live[c >> 5] >> (c & 31);
          if (w) return c + __ffs(w) - 1;
          c = (c | 31u) + 1;
        }
      }
      return min(c, nchunks);
    };
    if (MODE == kPull && threadIdx.x == 0 && nchunks) {     // bookkeeping: chunks of D_w that exist / that are read
      uint32_t read = nchunks;
      if (can_skip) {
        read = 0;
        for (uint32_t w = 0; w * 32 < nchunks; ++w) read += __popc(sh.live[w]);
      }
      atomicAdd(ws.stats + 3, (unsigned long long)nchunks);
      atomicAdd(ws.stats + 4, (unsigned long long)read);
    }
    uint32_t pc = 0, issued = 0;                          // thread 0: next chunk to ask for, chunks asked for
    if (threadIdx.x == 0) {
      pc = next_live(0);
      for (; issued < (uint32_t)R::kStages && pc < nchunks; ++issued, pc = next_live(pc + 1)) issue(pc, uses + issued);
    }
    uint32_t done = 0;
    for (uint32_t c = next_live(0); c < nchunks; c = next_live(c + 1), ++done) {
      const uint32_t use = uses + done, st = use % R::kStages;
      if (!mbar_wait(full + st, (use / R::kStages) & 1u)) *s_dead = 1;
      const uint32_t tl = c * kStageTiles + warp;          // this warp's tile among the full ones
      if (tl < nfull && !*s_dead) {
        const float* su = ring + (size_t)st * (R::kStageBytes / 4) + warp * kWarpTile;
        finish_full_tile_smem<MODE>(ws, a, sh, e0 + tl * kWarpTile, su, su + kStageFloats, L, slot0, lane, out);
      }
      __syncthreads();                                     // every warp is done reading this stage
      if (*s_dead) break;
      if (threadIdx.x == 0 && pc < nchunks) {
        issue(pc, uses + issued);
        ++issued;
        pc = next_live(pc + 1);
      }
    }
    if (*s_dead) break;
    uses += done;
    __syncthreads();
    flush_hist(sh.hist, ws.hist1 + (size_t)s * kBins1);
    __syncthreads();
  }
  if (*s_dead) {
    // a copy did not land in time: report, give the copies still in flight one more bounded wait, leave
    if (threadIdx.x == 0) {
      atomicMin(ws.status, kStatusTimeout);
      for (int st = 0; st < R::kStages; ++st) {
        mbar_wait(full + st, 0);
        mbar_wait(full + st, 1);
      }
    }
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

// Barrier among the CTAs of finalize (all resident: cooperative launch).  One arrival
// counter that only grows: the i-th barrier of a launch is passed when the counter has
// reached i*W (the stream pass that precedes every finalize launch clears the counter).
// Bounded: returns false, with the status word set, if the others do not arrive.
__device__ bool worker_barrier(uint32_t* sync, uint32_t W, int* status, int* s_ok, uint32_t& target) {
  target += W;
  __syncthreads();
  if (threadIdx.x == 0) {
    int ok = 1;
    __threadfence();
    atomicAdd(sync + kBarCount, 1u);
    uint32_t spins = 0;
    while ((int32_t)(ld_volatile(sync + kBarCount) - target) < 0) {
      if (++spins > kSpinLimit) {
        ok = 0;
        atomicMin(status, kStatusTimeout);
        break;
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
constexpr int kBatch = 8;       // independent loads a thread issues before using any (latency-bound loops)

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

// Walks the flat numbering: a thread (or a lane) owns consecutive flat candidates, finds
// the first one by binary search and then only steps.
struct Cursor {
  uint32_t part, slot, left;   // part of the current candidate, its slot, candidates left in that part (>= 1 if valid)
};
__device__ __forceinline__ Cursor cursor_at(const FinalizeShared& sh, uint32_t parts, uint32_t p) {
  Cursor c;
  c.slot = slot_of(sh, parts, p, &c.part);
  c.left = sh.pre_cands[c.part + 1] - p;
  return c;
}
// advance by n candidates; the caller never advances past the last candidate + 1
__device__ __forceinline__ void cursor_advance(const FinalizeShared& sh, uint32_t parts, Cursor& c, uint32_t n) {
  while (n >= c.left) {
    n -= c.left;
    do { ++c.part; } while (c.part < parts && sh.pre_cands[c.part + 1] == sh.pre_cands[c.part]);
    if (c.part >= parts) { c.left = 0xFFFFFFFFu; c.slot = 0; return; }   // ran off the end: never dereferenced
    c.slot = sh.slot0[c.part];
    c.left = sh.pre_cands[c.part + 1] - sh.pre_cands[c.part];
  }
  c.slot += n;
  c.left -= n;
}

template <int MODE>
__global__ void __maxnreg__(96) k_finalize(Workspace ws, SelArgs a) {
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

  // flat numbering of the candidates, and this thread's own candidates
  uint32_t parts = 0, C = 0, per_thread = 0, my_lo = 0, my_hi = 0;
  constexpr int kKeep = 8;            // candidates a thread keeps in registers between the phases
  uint32_t rkey[kKeep], ridx[kKeep];  // valid when per_thread <= kKeep
  uint32_t bar_target = 0;
  bool redo = false;
  for (int attempt = 0; attempt < 2; ++attempt) {
    if (redo) {
      // the guess was too high for some layer: take the bound that cannot fail from a histogram of
      // the whole input and repeat the stream pass, with the few CTAs this kernel has
      hist_all_tiles<MODE>(ws, a, in, cta, W, sh.stream.hist);
      if (!worker_barrier(ws.sync, W, ws.status, &sh.ok, bar_target)) return;
      for (uint32_t s = cta; s < S; s += W) {
        uint32_t bin, krem;
        uint32_t* h = ws.hist1 + (size_t)s * kBins1;
        const uint32_t k = ws.segs[s].k[PM];
        const uint32_t total = block_pick<kBins1>(h, k, bin, krem, sh.warp_scan, sh.res);
        uint32_t wbin = 0, wrem;
        const uint32_t want = max(k * kSpecFactor, k + kSpecSlack);
        if (total >= want) block_pick<kBins1>(h, want, wbin, wrem, sh.warp_scan, sh.res);
        if (threadIdx.x == 0) {
          ws.L_safe[s] = bin << 20;
          ws.L_wide[s] = wbin << 20;   // 0 (everything) when the layer has fewer than `want` entries
        }
        __syncthreads();
        for (int b = threadIdx.x; b < kBins1; b += kThreads) h[b] = 0;
      }
      if (cta == 0 && threadIdx.x == 0) ws.sync[kFail] = 0;
      if (!worker_barrier(ws.sync, W, ws.status, &sh.ok, bar_target)) return;
      stream_tiles<MODE>(ws, a, ws.L_safe, in, out, cta, W, sh.stream);
      if (!worker_barrier(ws.sync, W, ws.status, &sh.ok, bar_target)) return;
    }
    // flat numbering of the candidates (the stream pass is complete: an earlier kernel, or the barrier above)
    parts = ld_volatile(ws.sync + kParts);
    {
      constexpr int PER = kMaxGrid / kThreads;   // parts <= kMaxGrid
      uint32_t cnt[PER];
#pragma unroll
      for (int j = 0; j < PER; ++j) {
        const uint32_t p = j * kThreads + threadIdx.x;
        cnt[j] = p < parts ? __ldcg(ws.part_cands + p) : 0;
        if (p < parts) sh.slot0[p] = __ldcg(ws.part_slot0 + p);
      }
      unsigned long long carry = 0;
#pragma unroll
      for (int j = 0; j < PER; ++j) {
        if ((uint32_t)(j * kThreads) < parts) {   // CTA-uniform
          const uint32_t p = j * kThreads + threadIdx.x;
          unsigned long long total;
          const unsigned long long ex = block_excl_scan(cnt[j], sh.warp_scan, total) + carry;
          if (p < parts) sh.pre_cands[p] = (uint32_t)ex;
          carry += total;
        }
      }
      if (threadIdx.x == 0) sh.pre_cands[parts] = (uint32_t)carry;
      __syncthreads();
    }
    C = sh.pre_cands[parts];
    // every thread owns the flat candidates [my_lo, my_hi); when they are few it keeps them in registers
    per_thread = (C + nthreads - 1) / nthreads;
    my_lo = min(C, gthread * per_thread);
    my_hi = min(C, my_lo + per_thread);
    if (per_thread <= (uint32_t)kKeep && my_lo < my_hi) {
      Cursor cur = cursor_at(sh, parts, my_lo);
      float raw[kKeep];
#pragma unroll
      for (int u = 0; u < kKeep; ++u) {
        raw[u] = 0.f;
        ridx[u] = 0;
        if (my_lo + u < my_hi) {
          raw[u] = __ldcg(ws.cand_val + cur.slot);
          ridx[u] = __ldcg(ws.cand_idx + cur.slot);
          cursor_advance(sh, parts, cur, 1);
        }
      }
#pragma unroll
      for (int u = 0; u < kKeep; ++u) rkey[u] = key_of(raw[u]);
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
          } else if (redo || a.force_two_pass) {
            lbin = __ldcg(ws.L_wide + s) >> 20;   // known exactly from the histogram of the whole input
          } else {
            // fewer candidates than wished for and nothing known below the bound: lower it by half an octave
            const uint32_t used = a.L_in[s] >> 20;
            lbin = used > 4 ? used - 4 : 0;
          }
          __syncthreads();
          // A bound of zero makes every element of the layer a candidate (zeros included).  That is fine for a
          // layer not much larger than the wished-for number of candidates; for a large one, no bound at all is
          // the better advice: the next selection finds nothing, notices, and takes its bound from a histogram.
          const uint32_t layer_cap = (ws.segs[s].tile_end - ws.segs[s].tile_begin) * (uint32_t)kWarpTile;
          const bool flood = lbin == 0 && layer_cap / 8 > want;
          if (threadIdx.x == 0) a.L_next[s] = flood ? 0xFFFFFFFFu : lbin << 20;
        }
      }
      __syncthreads();
      for (int b = threadIdx.x; b < kBins1; b += kThreads) h[b] = 0;
    }
    if (!worker_barrier(ws.sync, W, ws.status, &sh.ok, bar_target)) return;
    if (redo || ld_volatile(ws.sync + kFail) == 0) break;
    redo = true;
  }

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
    if (S == 1) {
      for (int b = threadIdx.x; b < B; b += kThreads) sh.stream.hist[b] = 0;
      __syncthreads();
    }
    auto add_level = [&](uint32_t key, uint32_t idx) {
      const uint32_t seg = S > 1 ? seg_of(sv, idx) : 0;
      const uint32_t prefix = seg_smem ? sh.seg_a[seg] : __ldcg(&ws.sel[seg].prefix);
      if ((key >> SH) == prefix) {
        const uint32_t digit = (key >> (SH - 10)) & 1023u;
        if (S == 1) atomicAdd(sh.stream.hist + digit, 1u);       // one layer: CTA-private histogram first
        else atomicAdd(hist + (size_t)seg * B + digit, 1u);
      }
    };
    if (per_thread <= (uint32_t)kKeep) {
#pragma unroll
      for (int u = 0; u < kKeep; ++u)
        if (my_lo + u < my_hi) add_level(rkey[u], ridx[u]);
    } else if (my_lo < my_hi) {
      Cursor cur = cursor_at(sh, parts, my_lo);
      for (uint32_t p = my_lo; p < my_hi; p += kBatch) {
        // all loads of the batch are issued before any loaded value is touched (a use right
        // after its load would make the loads wait for one another)
        float raw[kBatch];
        uint32_t idx[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          raw[u] = 0.f;
          idx[u] = 0;
          if (p + u < my_hi) {
            raw[u] = __ldcg(ws.cand_val + cur.slot);
            if (S > 1) idx[u] = __ldcg(ws.cand_idx + cur.slot);
            cursor_advance(sh, parts, cur, 1);
          }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u)
          if (p + u < my_hi) add_level(key_of(raw[u]), idx[u]);
      }
    }
    if (S == 1) {
      __syncthreads();
      for (int b = threadIdx.x; b < B; b += kThreads) {
        const uint32_t v = sh.stream.hist[b];
        if (v) atomicAdd(hist + b, v);
      }
    }
    if (!worker_barrier(ws.sync, W, ws.status, &sh.ok, bar_target)) return;
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
    if (!worker_barrier(ws.sync, W, ws.status, &sh.ok, bar_target)) return;
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
  {
    auto add_count = [&](uint32_t key, uint32_t idx) {
      const uint32_t seg = S > 1 ? seg_of(sv, idx) : 0;
      const uint32_t T = seg_smem ? sh.seg_a[seg] : __ldcg(&ws.sel[seg].T);
      if (key >= T) {
        uint2* c = ws.tile_sel + tile_of(sv, seg, idx);
        atomicAdd(key > T ? &c->x : &c->y, 1u);
      }
    };
    if (per_thread <= (uint32_t)kKeep) {
#pragma unroll
      for (int u = 0; u < kKeep; ++u)
        if (my_lo + u < my_hi) add_count(rkey[u], ridx[u]);
    } else if (my_lo < my_hi) {
      Cursor cur = cursor_at(sh, parts, my_lo);
      for (uint32_t p = my_lo; p < my_hi; p += kBatch) {
        float raw[kBatch];
        uint32_t idx[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          raw[u] = 0.f;
          idx[u] = 0;
          if (p + u < my_hi) {
            raw[u] = __ldcg(ws.cand_val + cur.slot);
            idx[u] = __ldcg(ws.cand_idx + cur.slot);
            cursor_advance(sh, parts, cur, 1);
          }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u)
          if (p + u < my_hi) add_count(key_of(raw[u]), idx[u]);
      }
    }
  }
  if (!worker_barrier(ws.sync, W, ws.status, &sh.ok, bar_target)) return;

  // ---- scan over the tiles in index order: CTA c owns tiles [c*chunk, (c+1)*chunk) ----
  const uint32_t chunk_tiles = (ws.num_tiles + W - 1) / W;
  {
    const uint32_t t0 = min(ws.num_tiles, cta * chunk_tiles), t1 = min(ws.num_tiles, t0 + chunk_tiles);
    unsigned long long carry = 0;
    for (uint32_t base0 = t0; base0 < t1; base0 += kThreads * kBatch) {
      unsigned long long v[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const uint32_t t = base0 + u * kThreads + threadIdx.x;
        v[u] = 0;
        if (t < t1) {
          const uint2 c = __ldcg(ws.tile_sel + t);
          v[u] = ((unsigned long long)c.x << 32) | c.y;
        }
      }
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        if (base0 + u * kThreads < t1) {   // CTA-uniform
          const uint32_t t = base0 + u * kThreads + threadIdx.x;
          if (v[u]) ws.tile_sel[t] = make_uint2(0, 0);
          unsigned long long total;
          const unsigned long long ex = block_excl_scan(v[u], sh.warp_scan, total) + carry;
          if (t < t1) ws.tile_pre[t] = make_uint2((uint32_t)(ex >> 32), (uint32_t)ex);
          carry += total;
        }
      }
    }
    if (threadIdx.x == 0) ws.cta_tot[cta] = make_uint2((uint32_t)(carry >> 32), (uint32_t)carry);
  }
  if (!worker_barrier(ws.sync, W, ws.status, &sh.ok, bar_target)) return;

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
    // every warp owns a run of consecutive flat candidates, 32 per step
    const uint32_t gwarp = cta * kWarps + warp, nwarps = W * kWarps;
    const uint32_t per_warp = ((C + nwarps - 1) / nwarps + 31) / 32 * 32;
    const uint32_t w_lo = min(C, gwarp * per_warp), w_hi = min(C, w_lo + per_warp);
    Cursor cur;
    cur.part = 0; cur.slot = 0; cur.left = 0xFFFFFFFFu;
    if (w_lo + lane < w_hi) cur = cursor_at(sh, parts, w_lo + lane);
    // counts carried from the previous step for the tile its last lane was in
    uint32_t carry_gt = 0, carry_eq = 0, carry_tile = 0xFFFFFFFFu, carry_part = 0xFFFFFFFFu;
    for (uint32_t c0 = w_lo; c0 < w_hi; c0 += 32) {
      const uint32_t p = c0 + lane;
      const bool valid = p < w_hi;
      uint32_t part = 0xFFFFFFFEu, idx = 0, key = 0, seg = 0, tile = 0xFFFFFFFFu, T = 0, r = 0;
      float val = 0.f;
      if (valid) {
        part = cur.part;
        idx = __ldcg(ws.cand_idx + cur.slot);
        val = __ldcg(ws.cand_val + cur.slot);
        key = key_of(val);
        seg = S > 1 ? seg_of(sv, idx) : 0;
        tile = tile_of(sv, seg, idx);
        T = seg_smem ? sh.seg_a[seg] : __ldcg(&ws.sel[seg].T);
        r = seg_smem ? sh.seg_b[seg] : __ldcg(&ws.sel[seg].r);
        if (p + 32 < w_hi) cursor_advance(sh, parts, cur, 32);
      }
      const bool is_gt = valid && key > T, is_eq = valid && key == T;
      const uint32_t bgt = __ballot_sync(kFull, is_gt), beq = __ballot_sync(kFull, is_eq);
      // the candidates of one tile are consecutive: a lane starts a tile if its left neighbour is in another one
      const uint32_t left = __shfl_up_sync(kFull, tile, 1);
      const uint32_t heads = __ballot_sync(kFull, lane == 0 || left != tile);
      const int head = 31 - __clz(heads & (lt | (1u << lane)));       // first lane of my tile in this step
      const uint32_t mine = lt & ~((1u << head) - 1u);                  // lanes of my tile before me
      // what the tile of lane 0 holds in earlier slots
      const uint32_t tile0 = __shfl_sync(kFull, tile, 0), part0 = __shfl_sync(kFull, part, 0);
      uint32_t pre_gt = 0, pre_eq = 0;
      if (c0 != w_lo) {
        if (carry_tile == tile0 && carry_part == part0) {
          pre_gt = carry_gt;
          pre_eq = carry_eq;
        }
      } else {
        // first step of this warp: the tile may have begun in slots that belong to the previous warp
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
          pre_gt += __popc(__ballot_sync(kFull, same && k2 > T0));
          pre_eq += __popc(__ballot_sync(kFull, same && k2 == T0));
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
          gt_before += pre_gt;
          eq_before += pre_eq;
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
      // carry for the next step: counts of the tile that lane 31 is in (all lanes of a full step are valid)
      {
        const int head31 = 31 - __clz(heads);
        const uint32_t tail_lanes = ~((1u << head31) - 1u);
        carry_gt = __popc(bgt & tail_lanes) + (head31 == 0 ? pre_gt : 0u);
        carry_eq = __popc(beq & tail_lanes) + (head31 == 0 ? pre_eq : 0u);
        carry_tile = __shfl_sync(kFull, tile, 31);
        carry_part = __shfl_sync(kFull, part, 31);
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

// one CTA per layer (strided): L_safe = lower edge of the top-11-bit bin holding the k-th largest key,
// L_wide = the same for the max(3k, k+64)-th largest (the bound suggested for later selections)
template <int MODE>
__global__ void __launch_bounds__(kThreads) k_pick_lower(Workspace ws) {
  __shared__ unsigned long long s_warp[kWarps];
  __shared__ uint32_t s_res[2];
  constexpr int PM = MODE == kPull ? 1 : 0;
  for (uint32_t s = blockIdx.x; s < ws.num_segs; s += gridDim.x) {
    uint32_t bin, krem;
    uint32_t* h = ws.hist1 + (size_t)s * kBins1;
    const uint32_t k = ws.segs[s].k[PM];
    const uint32_t total = block_pick<kBins1>(h, k, bin, krem, s_warp, s_res);
    uint32_t wbin = 0, wrem;
    const uint32_t want = max(k * kSpecFactor, k + kSpecSlack);
    if (total >= want) block_pick<kBins1>(h, want, wbin, wrem, s_warp, s_res);
    if (threadIdx.x == 0) {
      ws.L_safe[s] = bin << 20;
      ws.L_wide[s] = wbin << 20;
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kBins1; b += kThreads) h[b] = 0;
  }
}

// ---- stand-alone stream pass with the carried bound -------------------------------
template <int MODE>
__global__ void __maxnreg__(64) k_stream(Workspace ws, SelArgs a) {
  extern __shared__ __align__(128) unsigned char dyn_smem[];   // the ring of stages
  __shared__ StreamShared sh;
  __shared__ __align__(8) uint64_t full[StreamRing<MODE>::kStages];
  __shared__ int s_dead;
  const float* in;
  float* out = nullptr;
  if (MODE == kPull) {
    in = a.D;
  } else {
    in = *a.u_cur_slot;
    out = *a.u_spare_slot;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) ws.sync[kBarCount] = 0;   // for the finalize launch that follows
  stream_tiles_tma<MODE>(ws, a, a.L_in, in, out, blockIdx.x, gridDim.x, sh, reinterpret_cast<float*>(dyn_smem), full,
                         &s_dead);
}

// ---- server apply ---------------------------------------------------------------
// Algorithm 2 lowers theta and every D_q by the decoded packet.  D_q is read only by worker
// q's pull, so the library keeps D_q lazily: an apply lowers theta at once and files the
// packet in a ring of recent packets; a pull of worker q first folds into D_q, in arrival
// order, the packets filed since D_q was last brought up to date.  Every D_q[i] sees the
// same subtractions in the same order as with an eager update, so the result is the same
// bit for bit, and each packet is folded into D_q while the entries it touches are hot
// instead of being scattered into all N vectors at once.
//
constexpr int kCatchGrid = 128;                             // CTAs of k_catch_up
constexpr uint32_t kCatchWarps = kCatchGrid * (kThreads / 32);
constexpr int kCatchBatch = 2;                              // entries per lane in flight per packet

struct PacketLog {
  uint32_t* idx;   // [ring][stride], each packet sorted by index
  float* val;      // [ring][stride]
  uint32_t stride; // entries between slots
  uint32_t cap;    // entries per packet
  uint32_t ring;   // slots
};

// theta -= packet, and a copy of the packet into slot `slot` of the log.
__global__ void __launch_bounds__(kThreads) k_apply_log(const uint32_t* __restrict__ idx,
                                                        const float* __restrict__ val, uint32_t count,
                                                        float* __restrict__ theta, uint64_t n, int* status,
                                                        PacketLog lg, uint32_t slot) {
  const uint32_t j = blockIdx.x * kThreads + threadIdx.x;
  if (j >= count) return;
  const uint32_t i = idx[j];
  const float v = val[j];
  lg.idx[(uint64_t)slot * lg.stride + j] = i;
  lg.val[(uint64_t)slot * lg.stride + j] = v;
  if (i >= n) {
    atomicMin(status, -2000);
    return;
  }
  theta[i] = __fsub_rn(theta[i], v);
}

// D -= packets first .. first + count - 1 of the log, in that order (count <= 64).  The index
// space is cut into kCatchWarps ranges holding equally many entries of the newest packet (the
// others are spread much alike); a warp owns one range, finds its part of every packet by
// binary search (packets are sorted), and takes the packets one after the other.  No two
// warps touch the same entry of D, so no atomics and no block-wide barriers are needed.
__global__ void __launch_bounds__(kThreads) k_catch_up(PacketLog lg, uint64_t first, uint32_t count,
                                                       float* __restrict__ D, uint32_t* __restrict__ blk_max,
                                                       uint64_t n) {
  const uint32_t lane = threadIdx.x & 31;
  const uint32_t w = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
  if (w >= kCatchWarps || count == 0) return;
  const uint32_t* ref = lg.idx + ((first + count - 1) % lg.ring) * (uint64_t)lg.stride;
  const uint32_t key_lo = w == 0 ? 0u : __ldcg(ref + (uint64_t)w * lg.cap / kCatchWarps);
  const uint32_t key_hi = w + 1 == kCatchWarps ? 0xFFFFFFFFu : __ldcg(ref + (uint64_t)(w + 1) * lg.cap / kCatchWarps);
  // positions of [key_lo, key_hi) in packet `lane` and in packet `lane + 32`
  uint32_t lo_r[2] = {0, 0}, hi_r[2] = {0, 0};
  {
    const uint32_t* a[2];
    uint32_t l0[2], r0[2], l1[2], r1[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t p = lane + 32 * h;
      a[h] = lg.idx + ((first + min(p, count - 1)) % lg.ring) * (uint64_t)lg.stride;
      l0[h] = l1[h] = 0;
      r0[h] = r1[h] = p < count ? lg.cap : 0;
    }
    for (uint32_t span = lg.cap; span > 0; span >>= 1) {  // enough halvings for a range of cap entries
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (l0[h] < r0[h]) {
          const uint32_t mid = (l0[h] + r0[h]) >> 1;
          if (__ldcg(a[h] + mid) < key_lo) l0[h] = mid + 1; else r0[h] = mid;
        }
        if (l1[h] < r1[h]) {
          const uint32_t mid = (l1[h] + r1[h]) >> 1;
          if (__ldcg(a[h] + mid) < key_hi) l1[h] = mid + 1; else r1[h] = mid;
        }
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      lo_r[h] = l0[h];
      hi_r[h] = l1[h];
    }
  }
  uint32_t ci[kCatchBatch], ni[kCatchBatch];
  float cv[kCatchBatch], nv[kCatchBatch];
  uint32_t lo = 0, hi = 0, nlo = 0, nhi = 0;
  const uint32_t* pi = nullptr;
  const float* pv = nullptr;
  const uint32_t* npi = nullptr;
  const float* npv = nullptr;
  auto fetch = [&](uint32_t p, uint32_t& flo, uint32_t& fhi, const uint32_t*& fpi, const float*& fpv,
                   uint32_t (&fi)[kCatchBatch], float (&fv)[kCatchBatch]) {
    const uint32_t a0 = __shfl_sync(0xFFFFFFFFu, lo_r[0], p & 31), a1 = __shfl_sync(0xFFFFFFFFu, lo_r[1], p & 31);
    const uint32_t b0 = __shfl_sync(0xFFFFFFFFu, hi_r[0], p & 31), b1 = __shfl_sync(0xFFFFFFFFu, hi_r[1], p & 31);
    flo = p < 32 ? a0 : a1;
    fhi = p < 32 ? b0 : b1;
    const uint64_t at = ((first + p) % lg.ring) * (uint64_t)lg.stride;
    fpi = lg.idx + at;
    fpv = lg.val + at;
#pragma unroll
    for (int e = 0; e < kCatchBatch; ++e) {
      const uint32_t j = flo + lane + 32 * e;
      const bool in = j < fhi;
      fi[e] = in ? __ldcg(fpi + j) : 0xFFFFFFFFu;
      fv[e] = in ? __ldcg(fpv + j) : 0.0f;
    }
  };
  fetch(0, lo, hi, pi, pv, ci, cv);
  for (uint32_t p = 0; p < count; ++p) {
    if (p + 1 < count) fetch(p + 1, nlo, nhi, npi, npv, ni, nv);
    for (uint32_t base = lo;;) {
      float d[kCatchBatch];
#pragma unroll
      for (int e = 0; e < kCatchBatch; ++e)
        if (ci[e] < n) d[e] = __ldcg(D + ci[e]);
#pragma unroll
      for (int e = 0; e < kCatchBatch; ++e)
        if (ci[e] < n) {
          const float r = __fsub_rn(d[e], cv[e]);
          __stcg(D + ci[e], r);
          atomicMax(blk_max + ci[e] / kWarpTile, key_of(r));   // keeps the block's bound an upper bound
        }
      base += 32 * kCatchBatch;
      if (base >= hi) break;
#pragma unroll
      for (int e = 0; e < kCatchBatch; ++e) {  // a range with more entries than one batch
        const uint32_t j = base + lane + 32 * e;
        const bool in = j < hi;
        ci[e] = in ? __ldcg(pi + j) : 0xFFFFFFFFu;
        cv[e] = in ? __ldcg(pv + j) : 0.0f;
      }
    }
    __syncwarp();  // orders this packet's stores before the next packet's loads within the warp
    lo = nlo;
    hi = nhi;
    pi = npi;
    pv = npv;
#pragma unroll
    for (int e = 0; e < kCatchBatch; ++e) {
      ci[e] = ni[e];
      cv[e] = nv[e];
    }
  }
}

// Eager form, for a packet that is not one of the library's own (any order of indices, any
// count): buffer q < N is D_q, buffer N is theta.  Indices of one packet are distinct, so every
// (buffer, entry) pair is touched by exactly one thread: plain load / subtract / store.
__global__ void __launch_bounds__(kThreads) k_scatter_sub(const uint32_t* __restrict__ idx,
                                                          const float* __restrict__ val, uint32_t count,
                                                          float* __restrict__ theta, float* __restrict__ D,
                                                          uint64_t d_stride, uint32_t num_workers, uint64_t n,
                                                          int* status, uint32_t* __restrict__ blk_max,
                                                          uint64_t blk_stride) {
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
  const float r = __fsub_rn(*p, v);
  *p = r;
  if (q < num_workers) atomicMax(blk_max + (uint64_t)q * blk_stride + i / kWarpTile, key_of(r));
}

}  // namespace dgs
