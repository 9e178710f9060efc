// Device code of the DGS push / apply / pull loop for sm_100a.
//
// Selection scheme (used for the worker's top-k of the velocity, Algorithm 3, and
// for the server's top-k of the model difference, Algorithm 2 / Eq. 6a):
//
//   stream pass   one read of the input.  Every element whose magnitude key is at
//                 least a per-layer lower bound L becomes a "candidate": (index,
//                 value) is appended, in index order, to the slot of its tile.
//                 Everything below L is final at once (the push writes t*(1/m)).
//   finalize      one cooperative kernel over the candidates only: three radix
//                 levels (11+10+10 bits of the key) find the exact k-th largest
//                 key T and the number r of entries equal to T that still fit;
//                 an ordered count/scan/emit writes the packet in index order.
//
// L is a guess carried from the worker's previous selection on that layer.  The
// guess is checked exactly (a layer needs at least k candidates); when it fails,
// or when there is no previous selection, finalize first runs a histogram pass
// over the whole input to get a bound that cannot fail, and repeats the stream
// pass itself.  The result never depends on the guess.
#pragma once
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dgs {
namespace cg = cooperative_groups;

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
constexpr int kMaxGrid = 2048;      // upper bound on the cooperative grid

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
  uint32_t pad[4];
};

enum Flag : int { kFlagFail = 0, kNumFlags = 4 };

struct Workspace {
  const Tile* tiles;
  const SegDesc* segs;
  uint32_t num_tiles, num_segs;
  uint32_t* cand_idx;   // [n]  candidates of tile t live at [tiles[t].start, +tile_count[t])
  float* cand_val;      // [n]
  uint32_t* tile_count; // [num_tiles]
  uint2* tile_pre;      // [num_tiles] CTA-local exclusive prefix of (key > T, key == T) counts
  uint2* cta_tot;       // [kMaxGrid]
  uint32_t* hist1;      // [S][kBins1]
  uint32_t* hist2;      // [S][kBins2]
  uint32_t* hist3;      // [S][kBins3]
  SegSel* sel;          // [S]
  uint32_t* L_safe;     // [S] bound from the whole-input histogram (two-pass route)
  uint32_t* flags;      // [kNumFlags]
  int* status;          // sticky device status word
  unsigned long long* stats;  // [0] single-pass selections, [1] two-pass selections
};

struct SelArgs {
  const float* grad;      // push: f32[n]
  float** u_cur_slot;     // push: device slot holding the worker's velocity pointer
  float** u_spare_slot;   // push: device slot holding the spare buffer pointer
  float* D;               // pull: D_w
  float* theta_local;     // pull: theta_w or null
  uint32_t* L_next;       // [S] lower bounds carried to this worker's next selection of this kind
  uint32_t* pkt_idx;
  float* pkt_val;
  uint32_t pkt_count;
  float m, lr, inv_m;
  int force_two_pass;
  int speculate;          // 0: never carry a bound (L_next is left alone)
};

__device__ __forceinline__ uint32_t key_of(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }
__device__ __forceinline__ uint32_t lanemask_lt() {
  uint32_t m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
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
// CTA `cta` of `G` handles a contiguous range of tiles, one tile per warp at a time.
template <int MODE>
__device__ void stream_tiles(const Workspace& ws, const SelArgs& a, const uint32_t* Larr,
                             const float* __restrict__ in, float* __restrict__ out, uint32_t cta, uint32_t G) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t t0 = (uint32_t)((uint64_t)cta * ws.num_tiles / G);
  const uint32_t t1 = (uint32_t)((uint64_t)(cta + 1) * ws.num_tiles / G);
  const uint32_t lt = lanemask_lt();
  for (uint32_t t = t0 + warp; t < t1; t += kWarps) {
    const Tile tile = ws.tiles[t];
    const uint32_t L = Larr[tile.seg];
    uint32_t* h1 = ws.hist1 + (size_t)tile.seg * kBins1;
    uint32_t running = 0;
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
      if (__any_sync(kFull, mask != 0)) {
#pragma unroll
        for (int j = 0; j < kVecIters; ++j) {
          const uint32_t mj = (mask >> (j * 4)) & 0xFu;
          if (!__any_sync(kFull, mj != 0)) continue;
          const uint32_t b0 = __ballot_sync(kFull, mj & 1u), b1 = __ballot_sync(kFull, mj & 2u);
          const uint32_t b2 = __ballot_sync(kFull, mj & 4u), b3 = __ballot_sync(kFull, mj & 8u);
          uint32_t pos = tile.start + running + __popc(b0 & lt) + __popc(b1 & lt) + __popc(b2 & lt) + __popc(b3 & lt);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            if ((mj >> c) & 1u) {
              const float v = x[4 * j + c];
              ws.cand_idx[pos] = tile.start + j * 128 + lane * 4 + c;
              ws.cand_val[pos] = v;
              atomicAdd(h1 + (key_of(v) >> 20), 1u);
              ++pos;
            }
          }
          running += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
        }
      }
    } else {
      for (uint32_t base = 0; base < tile.len; base += 32) {
        const uint32_t off = base + lane;
        const bool valid = off < tile.len;
        const uint32_t i = tile.start + off;
        float x = 0.f;
        bool cand = false;
        if (valid) {
          x = combine<MODE>(in[i], MODE != kPull ? a.grad[i] : 0.f, a.m, a.lr);
          cand = key_of(x) >= L;
          if (MODE != kPull) out[i] = cand ? x : unsent<MODE>(x, a.inv_m);
        }
        const uint32_t b = __ballot_sync(kFull, cand);
        if (cand) {
          const uint32_t pos = tile.start + running + __popc(b & lt);
          ws.cand_idx[pos] = i;
          ws.cand_val[pos] = x;
          atomicAdd(h1 + (key_of(x) >> 20), 1u);
        }
        running += __popc(b);
      }
    }
    if (lane == 0) ws.tile_count[t] = running;
  }
}

// ---- histogram of ALL elements (top 11 key bits), for the bound that cannot fail ----
__device__ __forceinline__ void flush_hist(uint32_t* s_hist, uint32_t* g_hist) {
  for (int b = threadIdx.x; b < kBins1; b += kThreads) {
    const uint32_t v = s_hist[b];
    if (v) {
      atomicAdd(g_hist + b, v);
      s_hist[b] = 0;
    }
  }
}

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
  const uint32_t t0 = (uint32_t)((uint64_t)cta * ws.num_tiles / G);
  const uint32_t t1 = (uint32_t)((uint64_t)(cta + 1) * ws.num_tiles / G);
  for (int b = threadIdx.x; b < kBins1; b += kThreads) s_hist[b] = 0;
  __syncthreads();
  if (t0 >= t1) return;
  uint32_t cur = ws.tiles[t0].seg;  // layer the shared histogram belongs to (CTA-uniform)
  for (uint32_t chunk = t0; chunk < t1; chunk += kWarps) {
    const uint32_t last = min(chunk + kWarps, t1) - 1;
    const uint32_t seg_lo = ws.tiles[chunk].seg, seg_hi = ws.tiles[last].seg;
    const uint32_t t = chunk + warp;
    Tile tile;
    tile.start = 0; tile.len = 0; tile.seg = 0xFFFF;
    if (t < t1) tile = ws.tiles[t];
    for (uint32_t s = seg_lo; s <= seg_hi; ++s) {
      if (s != cur) {
        __syncthreads();
        flush_hist(s_hist, ws.hist1 + (size_t)cur * kBins1);
        __syncthreads();
        cur = s;
      }
      if (t >= t1 || tile.seg != s) continue;
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
  }
  __syncthreads();
  flush_hist(s_hist, ws.hist1 + (size_t)cur * kBins1);
  __syncthreads();
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
    loc[j] = hist[top - j];
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

// ---- radix level over the candidates ---------------------------------------------
// LEVEL 2: candidates whose key bits 30..20 equal sel.prefix, digit = bits 19..10
// LEVEL 3: candidates whose key bits 30..10 equal sel.prefix, digit = bits  9..0
template <int LEVEL>
__device__ void hist_candidates(const Workspace& ws, uint32_t gwarp, uint32_t nwarps) {
  const int lane = threadIdx.x & 31;
  uint32_t* hist = LEVEL == 2 ? ws.hist2 : ws.hist3;
  constexpr int B = LEVEL == 2 ? kBins2 : kBins3;
  constexpr int SH = LEVEL == 2 ? 20 : 10;
  const uint32_t groups = (ws.num_tiles + 31) / 32;
  for (uint32_t g = gwarp; g < groups; g += nwarps) {
    const uint32_t t = g * 32 + lane;
    const uint32_t cnt = t < ws.num_tiles ? ws.tile_count[t] : 0;
    uint32_t nz = __ballot_sync(kFull, cnt != 0);
    while (nz) {
      const int src = __ffs(nz) - 1;
      nz &= nz - 1;
      const uint32_t c = __shfl_sync(kFull, cnt, src);
      const Tile tile = ws.tiles[g * 32 + src];
      const uint32_t prefix = ws.sel[tile.seg].prefix;
      for (uint32_t i = lane; i < c; i += 32) {
        const uint32_t key = key_of(ws.cand_val[tile.start + i]);
        if ((key >> SH) == prefix) atomicAdd(hist + (size_t)tile.seg * B + ((key >> (SH - 10)) & 1023u), 1u);
      }
    }
  }
}

// ---- finalize -------------------------------------------------------------------
template <int MODE>
__global__ void __launch_bounds__(kThreads, 2) k_finalize(Workspace ws, SelArgs a) {
  cg::grid_group grid = cg::this_grid();
  __shared__ uint32_t s_hist[kBins1];
  __shared__ unsigned long long s_warp[kWarps];
  __shared__ uint32_t s_res[2];
  __shared__ uint2 s_base[kMaxGrid];

  constexpr int PM = MODE == kPull ? 1 : 0;
  const uint32_t cta = blockIdx.x, G = gridDim.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t gwarp = cta * kWarps + warp, nwarps = G * kWarps;
  const uint32_t lt = lanemask_lt();

  // pointers are read once, before anything may exchange them
  const float* in = nullptr;
  float* out = nullptr;
  if (MODE == kPull) {
    in = a.D;
  } else {
    in = *a.u_cur_slot;
    out = *a.u_spare_slot;
  }
  grid.sync();

  bool two_pass = a.force_two_pass != 0;
  for (int attempt = 0; attempt < 2; ++attempt) {
    if (two_pass) {
      // bound that cannot fail: lower edge of the top-11-bit bin holding the k-th largest key
      hist_all_tiles<MODE>(ws, a, in, cta, G, s_hist);
      grid.sync();
      for (uint32_t s = cta; s < ws.num_segs; s += G) {
        uint32_t bin, krem;
        uint32_t* h = ws.hist1 + (size_t)s * kBins1;
        block_pick<kBins1>(h, ws.segs[s].k[PM], bin, krem, s_warp, s_res);
        if (threadIdx.x == 0) ws.L_safe[s] = bin << 20;
        for (int b = threadIdx.x; b < kBins1; b += kThreads) h[b] = 0;
      }
      if (cta == 0 && threadIdx.x == 0) ws.flags[kFlagFail] = 0;
      grid.sync();
      stream_tiles<MODE>(ws, a, ws.L_safe, in, out, cta, G);
      grid.sync();
    }
    // level 1: pick the bin of the k-th largest among the candidates; check the guess
    for (uint32_t s = cta; s < ws.num_segs; s += G) {
      uint32_t bin, krem;
      uint32_t* h = ws.hist1 + (size_t)s * kBins1;
      const uint32_t k = ws.segs[s].k[PM];
      const uint32_t total = block_pick<kBins1>(h, k, bin, krem, s_warp, s_res);
      if (total < k) {
        if (threadIdx.x == 0) atomicOr(ws.flags + kFlagFail, 1u);
      } else {
        if (threadIdx.x == 0) {
          ws.sel[s].prefix = bin;
          ws.sel[s].krem = krem;
        }
        if (a.speculate) {
          // bound for this worker's next selection on this layer
          const uint32_t want = max(k * kSpecFactor, k + kSpecSlack);
          uint32_t lbin, lrem;
          if (total >= want) {
            block_pick<kBins1>(h, want, lbin, lrem, s_warp, s_res);
          } else {
            const uint32_t used = (two_pass ? ws.L_safe[s] : a.L_next[s]) >> 20;
            lbin = used > 0 ? used - 1 : 0;
          }
          if (threadIdx.x == 0) a.L_next[s] = lbin << 20;
        }
      }
      __syncthreads();
      for (int b = threadIdx.x; b < kBins1; b += kThreads) h[b] = 0;
    }
    grid.sync();
    if (two_pass || ws.flags[kFlagFail] == 0) break;
    two_pass = true;  // the guess was too high somewhere: redo with a safe bound
  }

  // level 2
  hist_candidates<2>(ws, gwarp, nwarps);
  grid.sync();
  for (uint32_t s = cta; s < ws.num_segs; s += G) {
    uint32_t bin, krem;
    uint32_t* h = ws.hist2 + (size_t)s * kBins2;
    block_pick<kBins2>(h, ws.sel[s].krem, bin, krem, s_warp, s_res);
    __syncthreads();
    if (threadIdx.x == 0) {
      ws.sel[s].prefix = (ws.sel[s].prefix << 10) | bin;
      ws.sel[s].krem = krem;
    }
    for (int b = threadIdx.x; b < kBins2; b += kThreads) h[b] = 0;
  }
  grid.sync();
  // level 3
  hist_candidates<3>(ws, gwarp, nwarps);
  grid.sync();
  for (uint32_t s = cta; s < ws.num_segs; s += G) {
    uint32_t bin, krem;
    uint32_t* h = ws.hist3 + (size_t)s * kBins3;
    block_pick<kBins3>(h, ws.sel[s].krem, bin, krem, s_warp, s_res);
    __syncthreads();
    if (threadIdx.x == 0) {
      ws.sel[s].T = (ws.sel[s].prefix << 10) | bin;
      ws.sel[s].r = krem;
    }
    for (int b = threadIdx.x; b < kBins3; b += kThreads) h[b] = 0;
  }
  grid.sync();

  // ---- ordered count: per tile (#key > T, #key == T), CTA-local exclusive prefix ----
  const uint32_t t0 = (uint32_t)((uint64_t)cta * ws.num_tiles / G);
  const uint32_t t1 = (uint32_t)((uint64_t)(cta + 1) * ws.num_tiles / G);
  {
    unsigned long long carry = 0;
    for (uint32_t chunk = t0; chunk < t1; chunk += kThreads) {
      const uint32_t t = chunk + threadIdx.x;
      const uint32_t cnt = t < t1 ? ws.tile_count[t] : 0;
      uint32_t my_gt = 0, my_eq = 0;
      uint32_t nz = __ballot_sync(kFull, cnt != 0);
      while (nz) {
        const int src = __ffs(nz) - 1;
        nz &= nz - 1;
        const uint32_t c = __shfl_sync(kFull, cnt, src);
        const Tile tile = ws.tiles[chunk + warp * 32 + src];
        const uint32_t T = ws.sel[tile.seg].T;
        uint32_t gt = 0, eq = 0;
        for (uint32_t i = lane; i < c; i += 32) {
          const uint32_t key = key_of(ws.cand_val[tile.start + i]);
          gt += key > T;
          eq += key == T;
        }
        gt = __reduce_add_sync(kFull, gt);
        eq = __reduce_add_sync(kFull, eq);
        if (lane == src) {
          my_gt = gt;
          my_eq = eq;
        }
      }
      unsigned long long total;
      const unsigned long long v = ((unsigned long long)my_gt << 32) | my_eq;
      const unsigned long long ex = block_excl_scan(v, s_warp, total) + carry;
      if (t < t1) ws.tile_pre[t] = make_uint2((uint32_t)(ex >> 32), (uint32_t)ex);
      carry += total;
    }
    if (threadIdx.x == 0) ws.cta_tot[cta] = make_uint2((uint32_t)(carry >> 32), (uint32_t)carry);
  }
  grid.sync();

  // ---- emit: packet in index order, and the state updates that depend on selection ----
  {
    // exclusive prefix of the CTA totals (G <= kMaxGrid)
    unsigned long long carry = 0;
    for (uint32_t base = 0; base < G; base += kThreads) {
      const uint32_t c = base + threadIdx.x;
      unsigned long long v = 0;
      if (c < G) {
        const uint2 q = ws.cta_tot[c];
        v = ((unsigned long long)q.x << 32) | q.y;
      }
      unsigned long long total;
      const unsigned long long ex = block_excl_scan(v, s_warp, total) + carry;
      if (c < G) s_base[c] = make_uint2((uint32_t)(ex >> 32), (uint32_t)ex);
      carry += total;
    }
    __syncthreads();
    const uint2 my_base = s_base[cta];
    for (uint32_t chunk = t0 + warp * 32; chunk < t1; chunk += kThreads) {
      const uint32_t t = chunk + lane;
      const uint32_t cnt = t < t1 ? ws.tile_count[t] : 0;
      uint32_t nz = __ballot_sync(kFull, cnt != 0);
      while (nz) {
        const int src = __ffs(nz) - 1;
        nz &= nz - 1;
        const uint32_t c = __shfl_sync(kFull, cnt, src);
        const uint32_t tt = chunk + src;
        const Tile tile = ws.tiles[tt];
        const SegDesc sd = ws.segs[tile.seg];
        const uint32_t T = ws.sel[tile.seg].T, r = ws.sel[tile.seg].r;
        // counts before this tile, and before this tile's layer, in global tile order
        const uint2 pre = ws.tile_pre[tt];
        const uint32_t tb = sd.tile_begin;
        uint32_t owner = (uint32_t)(((uint64_t)tb * G) / ws.num_tiles);
        while (owner + 1 < G && (uint32_t)((uint64_t)(owner + 1) * ws.num_tiles / G) <= tb) ++owner;
        while (owner > 0 && (uint32_t)((uint64_t)owner * ws.num_tiles / G) > tb) --owner;
        const uint2 pre0 = ws.tile_pre[tb];
        const uint2 base0 = s_base[owner];
        uint32_t gt_run = (my_base.x + pre.x) - (base0.x + pre0.x);
        uint32_t eq_run = (my_base.y + pre.y) - (base0.y + pre0.y);
        for (uint32_t i0 = 0; i0 < c; i0 += 32) {
          const uint32_t i = i0 + lane;
          const bool valid = i < c;
          uint32_t idx = 0;
          float val = 0.f;
          uint32_t key = 0;
          if (valid) {
            idx = ws.cand_idx[tile.start + i];
            val = ws.cand_val[tile.start + i];
            key = key_of(val);
          }
          const bool is_gt = valid && key > T, is_eq = valid && key == T;
          const uint32_t bgt = __ballot_sync(kFull, is_gt), beq = __ballot_sync(kFull, is_eq);
          const uint32_t gt_before = gt_run + __popc(bgt & lt);
          const uint32_t eq_before = eq_run + __popc(beq & lt);
          const bool sel = is_gt || (is_eq && eq_before < r);
          if (valid) {
            if (sel) {
              const uint32_t pos = sd.pkt_off[PM] + gt_before + min(eq_before, r);
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
          gt_run += __popc(bgt);
          eq_run += __popc(beq);
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
    atomicAdd(ws.stats + (two_pass ? 1 : 0), 1ull);
  }
}

// ---- stand-alone stream pass with the carried bound -------------------------------
template <int MODE>
__global__ void __launch_bounds__(kThreads, 4) k_stream(Workspace ws, SelArgs a) {
  const float* in;
  float* out = nullptr;
  if (MODE == kPull) {
    in = a.D;
  } else {
    in = *a.u_cur_slot;
    out = *a.u_spare_slot;
  }
  stream_tiles<MODE>(ws, a, a.L_next, in, out, blockIdx.x, gridDim.x);
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
