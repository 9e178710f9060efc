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
constexpr uint32_t kSpecSlack = 64; // a carried bound aims at max(1.5 k, k + 64) candidates next time
constexpr int kMaxGrid = 512;       // upper bound on the grid of a stream pass (= parts of the candidate buffer)
constexpr int kMaxWorkers = 320;    // upper bound on the grid of finalize
constexpr uint32_t kSpinLimit = 1u << 22;  // bounded waits: give up and report after this many polls
constexpr int kStatusTimeout = -4;  // = DGS_ETIMEOUT
constexpr int kNumStats = 8;        // words of Workspace::stats (every owner of a Workspace provides that many)

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
  uint32_t neq;        // candidates with key == T
  uint32_t wrem;       // bound suggested for a later selection: rank of its entry inside the first-level bin of
                       // the k-th, when it lies in that bin (the second level then places it), else 0
};

// word indices in Workspace::sync
enum SyncWord : int { kBarCount = 0, kBarGen = 1, kDecision = 2, kFail = 3, kParts = 4, kPlanParts = 5, kNumSyncWords = 8 };

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
  // Pull, one layer: where the parts of the NEXT stream pass on this scratch set begin (tiles), planned by
  // finalize from what this pass cost each part; plan[parts] == num_tiles and plan_parts == parts mark it valid.
  uint32_t* plan;         // [kMaxGrid + 1], or null
  uint32_t* part_live;    // [kMaxGrid] chunks each part read in the last stream pass, or null
  const uint32_t* seg_off;   // [S+1] first element of each layer, and n
  const uint32_t* seg_tile0; // [S]   first tile of each layer
  uint2* cta_tot;         // [kMaxWorkers] (#key > T, #key == T) among the candidates of each CTA of finalize
  uint2* seg_start;       // [S] the same counted over all earlier layers
  uint32_t* hist1;        // [S][kBins1]
  uint32_t* hist2;        // [S][kBins2]
  uint32_t* hist3;        // [S][kBins3]
  SegSel* sel;            // [S]
  uint32_t* L_safe;       // [S] bound from the whole-input histogram (two-pass route)
  uint32_t* L_wide;       // [S] from the same histogram: the bound that admits about max(1.5 k, k+64) entries
  uint32_t* sync;         // [kNumSyncWords]
  int* status;            // sticky device status word
  // [kNumStats] counters: [0] single-pass selections, [1] two-pass selections, [2] candidates seen,
  // [3] chunks of difference vectors covered by the pulls' stream passes, [4] those of them read
  unsigned long long* stats;
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
  uint32_t phantom_workers;  // testing only: CTAs the finalize barrier waits for beyond those launched (0 in normal use)
  uint32_t spin_limit;    // polls after which a bounded wait gives up (0: kSpinLimit)
  int packet_format;      // 0: packets carry float32 values; 1: bfloat16; 2: binary16 (see round16)
};

__device__ __forceinline__ uint32_t key_of(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }
// A packet value in a 16-bit floating-point format, as the float32 number with that value (round to
// nearest, ties to even).  fmt 1: bfloat16 (8 exponent bits, 7 fraction bits).  fmt 2: IEEE binary16
// (5 exponent bits, 10 fraction bits, gradual underflow); a magnitude that would round beyond the largest
// finite binary16 number is sent as that number, 65504.  fmt 0: the value itself.  Inputs are finite.
__device__ __forceinline__ float round16(float x, int fmt) {
  if (fmt == 0) return x;
  const uint32_t b = __float_as_uint(x);
  uint32_t m = b & 0x7FFFFFFFu;
  if (fmt == 1) {
    m = (m + 0x7FFFu + ((m >> 16) & 1u)) & 0xFFFF0000u;
    if (m >= 0x7F800000u) m = 0x7F7F0000u;
  } else if (m >= 0x477FF000u) {          // 65520 and above
    m = 0x477FE000u;                      // 65504
  } else if (m >= 0x38800000u) {          // 2^-14 and above: 13 fraction bits go
    m = (m + 0xFFFu + ((m >> 13) & 1u)) & 0xFFFFE000u;
  } else {
    // steps of 2^-24 below 2^-14: the multiple nearest to |x| (scaling by powers of two is exact)
    const float scaled = __fmul_rn(__uint_as_float(m), 16777216.0f);
    const int whole = (int)scaled;        // truncation; scaled < 1024
    const float frac = __fsub_rn(scaled, (float)whole);
    const int up = (frac > 0.5f || (frac == 0.5f && (whole & 1))) ? 1 : 0;
    m = __float_as_uint(__fmul_rn((float)(whole + up), 1.0f / 16777216.0f));
  }
  return __uint_as_float(m | (b & 0x80000000u));
}
// candidates a carried bound should admit for a selection of k entries
__device__ __forceinline__ uint32_t spec_want(uint32_t k) { return max(k + k / 2, k + kSpecSlack); }
// A bound inside a bin of the first-level histogram (key bits 30..20 = bin): `need` of the bin's `pop`
// entries are wanted, counted from the largest down; the bin's keys are taken as evenly spread over
// [lo, hi), lo being the bin's lower edge or the bound that was in force if that cut the bin.  A quarter
// more than needed is admitted.  Only advice for a later selection: results never depend on it.
__device__ __forceinline__ uint32_t bound_inside_bin(uint32_t bin, uint32_t need, uint32_t pop, uint32_t floor_key) {
  const uint32_t hi = (bin + 1u) << 20;
  uint32_t lo = bin << 20;
  if (floor_key > lo && floor_key < hi) lo = floor_key;
  const uint32_t width = hi - lo;
  const float f = fminf(1.f, 1.25f * (float)need / (float)max(pop, 1u) + 0.02f);
  const uint32_t take = (uint32_t)ceilf(f * (float)width);
  return hi - min(width, take);
}
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
// Candidates are appended in INDEX ORDER: a CTA owns a contiguous range of tiles and a region
// of the candidate buffer; it takes its tiles in rounds of kWarps consecutive tiles (one per
// warp).  In a round every warp first counts the candidates of its tile, the counts are
// exchanged through shared memory, and each warp then writes its candidates behind those of the
// warps holding earlier tiles.  Read part after part, the candidate buffer therefore lists all
// candidates of the vector in ascending index order, which is what lets the finalize kernel
// number the selected ones with a plain prefix sum.
constexpr int kLiveWords = 128;     // one bit per stage-sized chunk of a CTA's share of a layer
struct StreamShared {
  uint32_t hist[kBins1];      // top 11 key bits of the candidates of the layer being processed
  uint32_t cursor;            // candidates appended by this CTA so far
  uint32_t wcnt[2][kWarps];   // candidates per warp of the current round (two rounds alternate)
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

// candidates of warps 0 .. warp-1 in this round, and of all warps
__device__ __forceinline__ uint32_t round_offset(const uint32_t* wcnt, int warp, uint32_t& total) {
  uint32_t before = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) {
    const uint32_t c = wcnt[w];
    if (w < warp) before += c;
    tot += c;
  }
  total = tot;
  return before;
}

// A full tile held in registers: x[16] are this lane's values (4 float4 at elements
// j*128 + lane*4 + c of the tile).  Returns the candidate mask; writes the new velocity (push).
template <int MODE>
__device__ __forceinline__ uint32_t tile_mask_regs(const SelArgs& a, uint32_t tile_start,
                                                   const float (&x)[4 * kVecIters], uint32_t L, int lane,
                                                   float* __restrict__ out) {
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
  return mask;
}

// Writes the candidates of a full tile (mask from tile_mask_*) from slot `base` on, in index
// order, and histograms their top key bits.  The cost is proportional to the candidates: one
// packed warp scan gives every lane the rank of its candidates (lane l holds elements
// j*128 + l*4 + c, order is j-major, so the four per-j counts travel as four bytes of one
// word), and a lane that has candidates walks its set bits.  value(off) returns element `off`.
template <typename ValueFn>
__device__ __forceinline__ void tile_emit(const Workspace& ws, StreamShared& sh, uint32_t tile_start, uint32_t mask,
                                          uint32_t base, int lane, ValueFn value) {
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
  const uint32_t t0 = tot & 0xFFu, t1 = (tot >> 8) & 0xFFu, t2 = (tot >> 16) & 0xFFu;
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
      const float v = value(off);
      ws.cand_idx[pos] = tile_start + off;
      ws.cand_val[pos] = v;
      atomicAdd(sh.hist + (key_of(v) >> 20), 1u);
    }
  }
}

// A ragged tile (first or last of a layer, fewer than kWarpTile elements or not 16-byte
// aligned): one element per lane and step, straight from global memory, at most 16 steps, the
// loads of eight steps in flight together.  Returns the candidate flags (one bit per step) and
// leaves the values of this lane's elements in x[step]; writes the new velocity (push).
constexpr int kRaggedSteps = kWarpTile / 32;
template <int MODE>
__device__ __forceinline__ uint32_t ragged_mask(const SelArgs& a, const Tile tile, uint32_t L, int lane,
                                                const float* __restrict__ in, float* __restrict__ out,
                                                float (&x)[kRaggedSteps]) {
  uint32_t flags = 0;
#pragma unroll
  for (int s0 = 0; s0 < kRaggedSteps; s0 += 8) {
    if (s0 * 32 < (int)tile.len) {   // warp-uniform
      float vu[8], vg[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t off = (s0 + j) * 32 + lane;
        vu[j] = 0.f;
        vg[j] = 0.f;
        if (off < tile.len) {
          vu[j] = in[tile.start + off];
          if (MODE != kPull) vg[j] = a.grad[tile.start + off];
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t off = (s0 + j) * 32 + lane;
        x[s0 + j] = 0.f;
        if (off < tile.len) {
          const float v = combine<MODE>(vu[j], vg[j], a.m, a.lr);
          const bool cand = key_of(v) >= L;
          if (MODE != kPull) out[tile.start + off] = cand ? v : unsent<MODE>(v, a.inv_m);
          if (cand) flags |= 1u << (s0 + j);
          x[s0 + j] = v;
        }
      }
    }
  }
  return flags;
}
// Writes its candidates from slot `base` on, in index order.
__device__ __forceinline__ void ragged_emit(const Workspace& ws, StreamShared& sh, const Tile tile, uint32_t flags,
                                            uint32_t base, int lane, uint32_t lt, const float (&x)[kRaggedSteps]) {
  if (!__any_sync(kFull, flags != 0)) return;
#pragma unroll
  for (int st = 0; st < kRaggedSteps; ++st) {
    if (st * 32 < (int)tile.len) {   // warp-uniform
      const bool cand = (flags >> st) & 1u;
      const uint32_t b = __ballot_sync(kFull, cand);
      if (cand) {
        const uint32_t pos = base + __popc(b & lt);
        ws.cand_idx[pos] = tile.start + st * 32 + lane;
        ws.cand_val[pos] = x[st];
        atomicAdd(sh.hist + (key_of(x[st]) >> 20), 1u);
      }
      base += __popc(b);
    }
  }
}

// CTA `cta` of `G` handles a contiguous range of tiles, kWarps consecutive tiles per round,
// layer by layer, so that the CTA's shared histogram always belongs to one layer; it is added
// to the global one when the CTA leaves the layer.  Loads go straight from global memory to
// registers (used where only a few CTAs run the pass).
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
  uint32_t cur = 0;      // candidates appended so far (the same in every thread)
  uint32_t round = 0;
  for (uint32_t s = seg_first; s <= seg_last; ++s) {
    const uint32_t a0 = max(t0, ws.segs[s].tile_begin), a1 = min(t1, ws.segs[s].tile_end);
    const uint32_t L = Larr[s];
    for (uint32_t tb = a0; tb < a1; tb += kWarps, ++round) {
      const uint32_t t = tb + warp;
      Tile tile;
      tile.start = 0; tile.len = 0; tile.seg = 0;
      float x[4 * kVecIters];
      uint32_t mask = 0;
      if (t < a1) {
        tile = ws.tiles[t];
        if (tile.len == kWarpTile) {
          load_tile_vec<MODE>(in, a.grad, tile.start, lane, a.m, a.lr, x);
          mask = tile_mask_regs<MODE>(a, tile.start, x, L, lane, out);
        } else {
          mask = ragged_mask<MODE>(a, tile, L, lane, in, out, x);
        }
      }
      const uint32_t count = __reduce_add_sync(kFull, (uint32_t)__popc(mask));
      if (lane == 0) sh.wcnt[round & 1][warp] = count;
      __syncthreads();
      uint32_t total;
      const uint32_t base = slot0 + cur + round_offset(sh.wcnt[round & 1], warp, total);
      cur += total;
      if (t < a1) {
        if (tile.len == kWarpTile) {
          tile_emit(ws, sh, tile.start, mask, base, lane, [&](uint32_t off) {
            // element off = j*128 + lane*4 + c is register 4*j + c of this lane
            const int e = (int)(((off >> 7) << 2) | (off & 3u));
            float v = x[0];
#pragma unroll
            for (int q = 1; q < 4 * kVecIters; ++q)
              if (q == e) v = x[q];
            return v;
          });
        } else {
          ragged_emit(ws, sh, tile, mask, base, lane, lt, x);
        }
      }
    }
    __syncthreads();
    flush_hist(sh.hist, ws.hist1 + (size_t)s * kBins1);
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    ws.part_cands[cta] = cur;
    ws.part_slot0[cta] = slot0;
  }
}

// Step one for a tile staged in shared memory (su: the tile of the state vector, sg: the tile
// of the gradient, push only): candidate mask, new velocity (push), block bound (pull).
template <int MODE>
__device__ __forceinline__ uint32_t tile_mask_smem(const SelArgs& a, uint32_t tile_start, const float* su,
                                                   const float* sg, uint32_t L, int lane, float* __restrict__ out) {
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
  return mask;
}

// ---- the same pass with TMA-staged tiles --------------------------------------------
// Full tiles are brought into a ring of shared-memory stages by bulk asynchronous copies
// (cp.async.bulk, completion counted on an mbarrier per stage), kStageTiles tiles of each
// input per stage, so that several stages are in flight while the warps work on one: the
// bytes in flight no longer depend on how many warps are waiting at a load.  One round of the
// ordered append = one stage; the barrier between counting and writing is also the one after
// which the stage of the round before is free, so a ring of kStages stages keeps kStages - 1
// of them in flight.
constexpr int kStageTiles = kWarps;                        // one tile per warp and stage
constexpr int kStageFloats = kStageTiles * kWarpTile;      // per input array
// The ring: three stages for a push (96 KB, two CTAs per SM, 128 KB of the SM's shared memory in flight),
// four for the staged form of a pull.
template <int MODE> struct StreamRing {
  static constexpr int kInputs = MODE == kPull ? 1 : 2;
  static constexpr int kStages = MODE == kPull ? 4 : 3;
  static constexpr int kStageBytes = kInputs * kStageFloats * 4;          // 16 KB per input
  static constexpr int kRingBytes = kStages * kStageBytes;
  static constexpr int kBytes = kRingBytes;
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
  static_assert(R::kStages >= 2, "the ring needs a stage in flight besides the one being read");
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t t0 = part_first_tile(cta, G, ws.num_tiles), t1 = part_first_tile(cta + 1, G, ws.num_tiles);
  if (MODE == kPull && ws.plan != nullptr && ld_volatile(ws.sync + kPlanParts) == G &&
      __ldcg(ws.plan + G) == ws.num_tiles) {
    // boundaries planned by the finalize of the previous selection on this scratch set
    t0 = __ldcg(ws.plan + cta);
    t1 = __ldcg(ws.plan + cta + 1);
  }
  uint32_t live_read = 0;   // thread 0: chunks this part reads
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
      if (MODE == kPull && ws.part_live != nullptr) ws.part_live[cta] = 0;
    }
    return;
  }
  const uint32_t slot0 = ws.tiles[t0].start;
  const uint32_t seg_first = ws.tiles[t0].seg, seg_last = ws.tiles[t1 - 1].seg;
  uint32_t uses = 0;  // stage uses so far (same in every thread): stage = use % kStages, parity = (use / kStages) & 1
  uint32_t cur = 0;   // candidates appended so far (same in every thread)
  for (uint32_t s = seg_first; s <= seg_last; ++s) {
    const uint32_t a0 = max(t0, ws.segs[s].tile_begin), a1 = min(t1, ws.segs[s].tile_end);
    const uint32_t L = Larr[s];
    // only the first and the last tile of a layer can be ragged
    const bool head = ws.tiles[a0].len != kWarpTile;
    const bool tail = (a1 - 1 > a0 || !head) && ws.tiles[a1 - 1].len != kWarpTile;
    const uint32_t f0 = a0 + (head ? 1u : 0u), f1 = a1 - (tail ? 1u : 0u);   // full tiles [f0, f1)
    // a ragged tile is one warp's work; the warp tells the others how many candidates it appended
    auto ragged = [&](uint32_t t) {
      if (warp == 0) {
        const Tile tile = ws.tiles[t];
        float x[kRaggedSteps];
        const uint32_t flags = ragged_mask<MODE>(a, tile, L, lane, in, out, x);
        const uint32_t count = __reduce_add_sync(kFull, (uint32_t)__popc(flags));
        ragged_emit(ws, sh, tile, flags, slot0 + cur, lane, lt, x);
        if (lane == 0) sh.cursor = count;
      }
      __syncthreads();
      cur += sh.cursor;
      __syncthreads();
    };
    if (head) ragged(a0);
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
      live_read += read;
    }
    uint32_t pc = 0, issued = 0;                          // thread 0: next chunk to ask for, chunks asked for
    if (threadIdx.x == 0) {
      pc = next_live(0);
      for (; issued < (uint32_t)R::kStages - 1 && pc < nchunks; ++issued, pc = next_live(pc + 1))
        issue(pc, uses + issued);
    }
    uint32_t done = 0;
    for (uint32_t c = next_live(0); c < nchunks; c = next_live(c + 1), ++done) {
      const uint32_t use = uses + done, st = use % R::kStages;
      const bool landed = mbar_wait(full + st, (use / R::kStages) & 1u);
      if (!landed) *s_dead = 1;
      const uint32_t tl = c * kStageTiles + warp;          // this warp's tile among the full ones
      const float* su = ring + (size_t)st * (R::kStageBytes / 4) + warp * kWarpTile;
      uint32_t mask = 0;
      if (tl < nfull && landed) mask = tile_mask_smem<MODE>(a, e0 + tl * kWarpTile, su, su + kStageFloats, L, lane, out);
      const uint32_t count = __reduce_add_sync(kFull, (uint32_t)__popc(mask));
      if (lane == 0) sh.wcnt[use & 1][warp] = count;
      __syncthreads();   // the counts of this round are known, and every warp has left the stage of the round before
      if (*s_dead) break;
      if (threadIdx.x == 0 && pc < nchunks) {              // into the stage of the round before
        issue(pc, uses + issued);
        ++issued;
        pc = next_live(pc + 1);
      }
      uint32_t total;
      const uint32_t base = slot0 + cur + round_offset(sh.wcnt[use & 1], warp, total);
      cur += total;
      tile_emit(ws, sh, e0 + tl * kWarpTile, mask, base, lane, [&](uint32_t off) {
        return combine<MODE>(su[off], MODE != kPull ? su[kStageFloats + off] : 0.f, a.m, a.lr);
      });
    }
    if (*s_dead) break;
    uses += done;
    __syncthreads();   // every warp has left the last stage (the next layer's first copies go anywhere in the ring)
    if (tail) ragged(a1 - 1);
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
    ws.part_cands[cta] = cur;
    ws.part_slot0[cta] = slot0;
    if (MODE == kPull && ws.part_live != nullptr) ws.part_live[cta] = live_read;
  }
}

// ---- the pull's pass without a staging ring ------------------------------------------
// A pull of one worker among many reads only the chunks of D_w whose block bounds admit a
// candidate -- a small part of the vector, a few chunks per CTA -- while the push passes of
// later events stream beside it and need the SMs' shared memory for their own rings.  This
// form of the pass therefore holds no ring: a warp loads its tile of the next chunk to be read
// straight into registers while the CTA finishes the chunk before, so one chunk is in flight
// per CTA, and the CTA keeps only its histogram in shared memory.  Candidates, bounds, plan and
// counters are exactly those of the staged form.
__device__ __forceinline__ void load_tile_raw(const float* __restrict__ in, uint32_t start, int lane,
                                              float (&x)[4 * kVecIters]) {
  const float4* pa = reinterpret_cast<const float4*>(in + start) + lane;
#pragma unroll
  for (int j = 0; j < kVecIters; ++j) {
    const float4 v = __ldcs(pa + j * 32);
    x[4 * j + 0] = v.x;
    x[4 * j + 1] = v.y;
    x[4 * j + 2] = v.z;
    x[4 * j + 3] = v.w;
  }
}

__device__ void pull_tiles_light(const Workspace& ws, const SelArgs& a, const uint32_t* Larr,
                                 const float* __restrict__ in, uint32_t cta, uint32_t G, StreamShared& sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t t0 = part_first_tile(cta, G, ws.num_tiles), t1 = part_first_tile(cta + 1, G, ws.num_tiles);
  if (ws.plan != nullptr && ld_volatile(ws.sync + kPlanParts) == G && __ldcg(ws.plan + G) == ws.num_tiles) {
    // boundaries planned by the finalize of the previous selection on this scratch set
    t0 = __ldcg(ws.plan + cta);
    t1 = __ldcg(ws.plan + cta + 1);
  }
  uint32_t live_read = 0;   // thread 0: chunks this part reads
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
      if (ws.part_live != nullptr) ws.part_live[cta] = 0;
    }
    return;
  }
  const uint32_t slot0 = ws.tiles[t0].start;
  const uint32_t seg_first = ws.tiles[t0].seg, seg_last = ws.tiles[t1 - 1].seg;
  uint32_t cur = 0;     // candidates appended so far (same in every thread)
  uint32_t round = 0;
  for (uint32_t s = seg_first; s <= seg_last; ++s) {
    const uint32_t a0 = max(t0, ws.segs[s].tile_begin), a1 = min(t1, ws.segs[s].tile_end);
    const uint32_t L = Larr[s];
    const bool head = ws.tiles[a0].len != kWarpTile;
    const bool tail = (a1 - 1 > a0 || !head) && ws.tiles[a1 - 1].len != kWarpTile;
    const uint32_t f0 = a0 + (head ? 1u : 0u), f1 = a1 - (tail ? 1u : 0u);   // full tiles [f0, f1)
    auto ragged = [&](uint32_t t) {
      if (warp == 0) {
        const Tile tile = ws.tiles[t];
        float x[kRaggedSteps];
        const uint32_t flags = ragged_mask<kPull>(a, tile, L, lane, in, nullptr, x);
        const uint32_t count = __reduce_add_sync(kFull, (uint32_t)__popc(flags));
        ragged_emit(ws, sh, tile, flags, slot0 + cur, lane, lt, x);
        if (lane == 0) sh.cursor = count;
      }
      __syncthreads();
      cur += sh.cursor;
      __syncthreads();
    };
    if (head) ragged(a0);
    const uint32_t nfull = f1 > f0 ? f1 - f0 : 0;
    const uint32_t nchunks = (nfull + kStageTiles - 1) / kStageTiles;
    const uint32_t e0 = nfull ? ws.tiles[f0].start : 0;   // first element of the full tiles (multiple of kWarpTile)
    // a chunk all of whose blocks have a bound below L holds no candidate and is not read
    const bool can_skip = a.blk_max != nullptr && L > 0 && nchunks <= kLiveWords * 32;
    if (can_skip) {
      for (uint32_t base = warp * 32; base < nchunks; base += kWarps * 32) {
        const uint32_t c = base + lane;
        bool live = false;
        if (c < nchunks) {
          const uint32_t tiles_here = min((uint32_t)kStageTiles, nfull - c * kStageTiles);
          const uint32_t* bm = a.blk_max + e0 / kWarpTile + c * kStageTiles;
          uint32_t top = 0;
          if (tiles_here == kStageTiles && (reinterpret_cast<uintptr_t>(bm) & 15u) == 0) {
            const uint4 q0 = __ldcg(reinterpret_cast<const uint4*>(bm)), q1 = __ldcg(reinterpret_cast<const uint4*>(bm) + 1);
            top = max(max(max(q0.x, q0.y), max(q0.z, q0.w)), max(max(q1.x, q1.y), max(q1.z, q1.w)));
          } else {
            for (uint32_t j = 0; j < tiles_here; ++j) top = max(top, __ldcg(bm + j));
          }
          live = top >= L;
        }
        const uint32_t word = __ballot_sync(kFull, live);
        if (lane == 0) sh.live[base / 32] = word;
      }
      __syncthreads();
    }
    auto next_live = [&](uint32_t c) -> uint32_t {       // first chunk >= c that is read, nchunks if none
      while (can_skip && c < nchunks) {
        const uint32_t w = sh.live[c >> 5] >> (c & 31);
        if (w) return c + __ffs(w) - 1;
        c = (c | 31u) + 1;
      }
      return min(c, nchunks);
    };
    if (threadIdx.x == 0 && nchunks) {     // bookkeeping: chunks of D_w that exist / that are read
      uint32_t read = nchunks;
      if (can_skip) {
        read = 0;
        for (uint32_t w = 0; w * 32 < nchunks; ++w) read += __popc(sh.live[w]);
      }
      atomicAdd(ws.stats + 3, (unsigned long long)nchunks);
      atomicAdd(ws.stats + 4, (unsigned long long)read);
      live_read += read;
    }
    float x[4 * kVecIters], xn[4 * kVecIters];
    uint32_t c = next_live(0);
    if (c < nchunks && c * kStageTiles + warp < nfull) load_tile_raw(in, e0 + (c * kStageTiles + warp) * kWarpTile, lane, x);
    while (c < nchunks) {
      const uint32_t cn = next_live(c + 1);
      const uint32_t tl = c * kStageTiles + warp;          // this warp's tile among the full ones
      const uint32_t tile_start = e0 + tl * kWarpTile;
      uint32_t mask = 0;
      if (tl < nfull) {
        uint32_t top = 0;
#pragma unroll
        for (int e = 0; e < 4 * kVecIters; ++e) {
          const uint32_t key = key_of(x[e]);
          top = max(top, key);
          if (key >= L) mask |= 1u << e;
        }
        if (a.blk_max != nullptr) {
          // the tile is a whole block: its bound becomes exact again (entries sent later only lower it)
          top = __reduce_max_sync(kFull, top);
          if (lane == 0) a.blk_max[tile_start / kWarpTile] = top;
        }
      }
      const uint32_t count = __reduce_add_sync(kFull, (uint32_t)__popc(mask));
      if (lane == 0) sh.wcnt[round & 1][warp] = count;
      // the next chunk is on its way while this one is written out
      if (cn < nchunks && cn * kStageTiles + warp < nfull)
        load_tile_raw(in, e0 + (cn * kStageTiles + warp) * kWarpTile, lane, xn);
      __syncthreads();
      uint32_t total;
      const uint32_t base = slot0 + cur + round_offset(sh.wcnt[round & 1], warp, total);
      cur += total;
      if (tl < nfull)
        tile_emit(ws, sh, tile_start, mask, base, lane, [&](uint32_t off) {
          // element off = j*128 + lane*4 + c is register 4*j + c of this lane
          const int e = (int)(((off >> 7) << 2) | (off & 3u));
          float v = x[0];
#pragma unroll
          for (int q = 1; q < 4 * kVecIters; ++q)
            if (q == e) v = x[q];
          return v;
        });
#pragma unroll
      for (int e = 0; e < 4 * kVecIters; ++e) x[e] = xn[e];
      c = cn;
      ++round;
    }
    __syncthreads();
    if (tail) ragged(a1 - 1);
    flush_hist(sh.hist, ws.hist1 + (size_t)s * kBins1);
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    ws.part_cands[cta] = cur;
    ws.part_slot0[cta] = slot0;
    if (ws.part_live != nullptr) ws.part_live[cta] = live_read;
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
__device__ bool worker_barrier(uint32_t* sync, uint32_t W, int* status, int* s_ok, uint32_t& target,
                               uint32_t limit = kSpinLimit) {
  target += W;
  __syncthreads();
  if (threadIdx.x == 0) {
    int ok = 1;
    __threadfence();
    atomicAdd(sync + kBarCount, 1u);
    uint32_t spins = 0;
    while ((int32_t)(ld_volatile(sync + kBarCount) - target) < 0) {
      if (++spins > limit) {
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
// consecutive slots from part_slot0[p] on.  Parts follow one another in index order and every
// part lists its candidates in index order, so the flat numbering is the index order of all
// candidates.  Every thread owns a run of consecutive flat candidates (kept in registers when
// they are few) for all phases:
//   levels 2 and 3   histograms of the next 10 + 10 key bits among the candidates that share the
//                    bits fixed so far  ->  exact k-th largest key T and tie quota r per layer
//   count            (key > T, key == T) per thread, prefix sums inside the CTA, totals per CTA
//   emit             a candidate's rank among the selected ones of its layer follows from the
//                    prefix sums (layers are consecutive in the flat order and layer s selects
//                    exactly k_s entries)  ->  packet in index order, state updates
// With one layer every CTA works out the picks itself from the shared histograms, which leaves
// three grid-wide barriers; with several layers the picks are spread over the CTAs.
constexpr int kSegCap = 1024;  // layers whose tables fit in shared memory; more fall back to global reads
constexpr int kBatch = 8;       // independent loads a thread issues before using any (latency-bound loops)

struct FinalizeShared {
  StreamShared stream;                 // redo of the passes (guess failed); its histogram also serves levels 2 and 3
  unsigned long long warp_scan[kWarps];
  uint32_t res[2];
  int ok;
  uint32_t pre_cands[kMaxGrid + 1];    // exclusive prefix of part_cands
  uint32_t slot0[kMaxGrid];            // first slot of each part
};
// Per-layer tables of finalize live in dynamic shared memory, sized by the number of layers S (up
// to kSegCap layers; with more, the kernel reads the tables from global memory and needs none):
//   uint2 seg_start[S]   (key > T, key == T) candidates of all earlier layers
//   u32 seg_off[S + 1]   first element of each layer, and n
//   u32 seg_a[S]         per-layer parameter of the current phase (prefix, or T)
//   u32 seg_b[S]         second one (r)
__host__ __device__ inline uint32_t finalize_dyn_bytes(uint32_t S) {
  return S <= (uint32_t)kSegCap ? 20u * S + 8u : 0u;
}

// layer that holds element i: last s with off[s] <= i
__device__ __forceinline__ uint32_t seg_of(const uint32_t* off, uint32_t S, uint32_t i) {
  uint32_t lo = 0, hi = S - 1;
  while (lo < hi) {
    const uint32_t mid = (lo + hi + 1) >> 1;
    if (off[mid] <= i) lo = mid; else hi = mid - 1;
  }
  return lo;
}
// The same for a thread that visits candidates in index order: consecutive candidates mostly lie in the
// same layer, so the layer found last is tried first and the search is only made when it does not hold i.
__device__ __forceinline__ uint32_t seg_near(const uint32_t* off, uint32_t S, uint32_t i, uint32_t& last) {
  if (i < off[last] || i >= off[last + 1]) last = seg_of(off, S, i);
  return last;
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

// Walks the flat numbering: a thread owns consecutive flat candidates, finds the first one by
// binary search and then only steps.
struct Cursor {
  uint32_t part, slot, left;   // part of the current candidate, its slot, candidates left in that part (>= 1 if valid)
};
__device__ __forceinline__ Cursor cursor_at(const FinalizeShared& sh, uint32_t parts, uint32_t p) {
  Cursor c;
  c.slot = slot_of(sh, parts, p, &c.part);
  c.left = sh.pre_cands[c.part + 1] - p;
  return c;
}
// advance by n candidates; the caller never dereferences a cursor that ran past the last candidate
__device__ __forceinline__ void cursor_advance(const FinalizeShared& sh, uint32_t parts, Cursor& c, uint32_t n) {
  while (n >= c.left) {
    n -= c.left;
    do { ++c.part; } while (c.part < parts && sh.pre_cands[c.part + 1] == sh.pre_cands[c.part]);
    if (c.part >= parts) { c.left = 0xFFFFFFFFu; c.slot = 0; return; }   // ran off the end
    c.slot = sh.slot0[c.part];
    c.left = sh.pre_cands[c.part + 1] - sh.pre_cands[c.part];
  }
  c.slot += n;
  c.left -= n;
}

// 64 registers a thread: finalize runs beside two CTAs of a push pass on an SM, which leave it that many
template <int MODE>
__global__ void __maxnreg__(64) k_finalize(Workspace ws, SelArgs a) {
  __shared__ FinalizeShared sh;
  extern __shared__ __align__(16) unsigned char fin_dyn[];   // finalize_dyn_bytes(S) bytes

  constexpr int PM = MODE == kPull ? 1 : 0;
  const uint32_t cta = blockIdx.x, W = gridDim.x, S = ws.num_segs;
  const uint32_t gthread = cta * kThreads + threadIdx.x, nthreads = W * kThreads;
  // the barrier counts W arrivals; a test can make it wait for CTAs that do not exist, with a short limit,
  // to see the bounded wait give up (every CTA then leaves with DGS_ETIMEOUT in the status word)
  const uint32_t Wb = W + a.phantom_workers, spin_limit = a.spin_limit ? a.spin_limit : kSpinLimit;

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
  uint2* const sm_seg_start = reinterpret_cast<uint2*>(fin_dyn);
  uint32_t* const sm_seg_off = reinterpret_cast<uint32_t*>(fin_dyn + 8u * S);
  uint32_t* const sm_seg_a = sm_seg_off + S + 1;
  uint32_t* const sm_seg_b = sm_seg_a + S;
  if (seg_smem)
    for (uint32_t s = threadIdx.x; s <= S; s += kThreads) sm_seg_off[s] = ws.seg_off[s];
  const uint32_t* const seg_off = seg_smem ? sm_seg_off : ws.seg_off;
  __syncthreads();

  // flat numbering of the candidates, and this thread's own candidates
  uint32_t parts = 0, C = 0, per_thread = 0, my_lo = 0, my_hi = 0;
  constexpr int kKeep = 8;            // candidates a thread keeps in registers between the phases
  float rraw[kKeep];
  uint32_t ridx[kKeep];               // valid when per_thread <= kKeep
  uint32_t bar_target = 0;
  uint32_t one_prefix = 0, one_krem = 0;   // S == 1: the layer's selection state, the same in every thread of the grid
  uint32_t one_wrem = 0;                   // S == 1, CTA 0: SegSel::wrem of the layer
  bool redo = false;
  for (int attempt = 0; attempt < 2; ++attempt) {
    if (redo) {
      // the guess was too high for some layer: take the bound that cannot fail from a histogram of
      // the whole input and repeat the stream pass, with the few CTAs this kernel has
      hist_all_tiles<MODE>(ws, a, in, cta, W, sh.stream.hist);
      if (!worker_barrier(ws.sync, Wb, ws.status, &sh.ok, bar_target, spin_limit)) return;
      for (uint32_t s = cta; s < S; s += W) {
        uint32_t bin, krem;
        uint32_t* h = ws.hist1 + (size_t)s * kBins1;
        const uint32_t k = ws.segs[s].k[PM];
        const uint32_t total = block_pick<kBins1>(h, k, bin, krem, sh.warp_scan, sh.res);
        uint32_t wbin = 0, wrem = 0;
        const uint32_t want = spec_want(k);
        if (total >= want) block_pick<kBins1>(h, want, wbin, wrem, sh.warp_scan, sh.res);
        if (threadIdx.x == 0) {
          ws.L_safe[s] = bin << 20;
          // 0 (everything) when the layer has fewer than `want` entries
          ws.L_wide[s] = total >= want ? bound_inside_bin(wbin, wrem, __ldcg(h + wbin), 0u) : 0u;
        }
        __syncthreads();
        for (int b = threadIdx.x; b < kBins1; b += kThreads) h[b] = 0;
      }
      if (cta == 0 && threadIdx.x == 0) ws.sync[kFail] = 0;
      if (!worker_barrier(ws.sync, Wb, ws.status, &sh.ok, bar_target, spin_limit)) return;
      stream_tiles<MODE>(ws, a, ws.L_safe, in, out, cta, W, sh.stream);
      if (!worker_barrier(ws.sync, Wb, ws.status, &sh.ok, bar_target, spin_limit)) return;
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
#pragma unroll
      for (int u = 0; u < kKeep; ++u) {
        rraw[u] = 0.f;
        ridx[u] = 0;
        if (my_lo + u < my_hi) {
          rraw[u] = __ldcg(ws.cand_val + cur.slot);
          ridx[u] = __ldcg(ws.cand_idx + cur.slot);
          cursor_advance(sh, parts, cur, 1);
        }
      }
    }
    // level 1: the bin of the k-th largest among the candidates; checks the guess, suggests the next one
    bool failed = false;
    const bool everyone_picks = S == 1;   // one layer: every CTA reads the histogram itself, no barrier needed
    for (uint32_t s = everyone_picks ? 0 : cta; s < S; s += everyone_picks ? 1 : W) {
      uint32_t bin, krem;
      uint32_t* h = ws.hist1 + (size_t)s * kBins1;
      const uint32_t k = ws.segs[s].k[PM];
      const uint32_t total = block_pick<kBins1>(h, k, bin, krem, sh.warp_scan, sh.res);
      const bool owner = !everyone_picks || cta == 0;
      if (total < k) {
        failed = true;
        if (owner && threadIdx.x == 0) atomicOr(ws.sync + kFail, 1u);
      } else {
        one_prefix = bin;
        one_krem = krem;
        if (owner && threadIdx.x == 0) {
          ws.sel[s].prefix = bin;
          ws.sel[s].krem = krem;
          ws.sel[s].wrem = 0;
          atomicAdd(ws.stats + 2, (unsigned long long)total);
        }
        one_wrem = 0;
        if (owner && a.speculate) {
          // bound suggested for a later selection on this layer
          const uint32_t want = spec_want(k);
          uint32_t lbin, lrem;
          uint32_t lkey;   // the bound itself
          if (total >= want) {
            block_pick<kBins1>(h, want, lbin, lrem, sh.warp_scan, sh.res);
            const uint32_t in_force = (redo || a.force_two_pass) ? __ldcg(ws.L_safe + s) : a.L_in[s];
            lkey = bound_inside_bin(lbin, lrem, __ldcg(h + lbin), in_force);
            // Inside the bin of the k-th the keys are anything but evenly spread where a push has run for a
            // while: what was never sent piles up right below the k-th, what lies above it is a thin tail, and
            // a bound interpolated from the top of the bin lands in the tail (the next selection then finds
            // fewer than k candidates and starts over).  The second level counts that bin in 1024 parts.
            if (lbin == bin && bin > 0) {
              const uint32_t roomy = lrem + want / 16;          // a little beyond, if the bin holds that many
              one_wrem = roomy <= __ldcg(h + bin) ? roomy : lrem;
              if (threadIdx.x == 0) ws.sel[s].wrem = one_wrem;
            }
          } else if (redo || a.force_two_pass) {
            lkey = __ldcg(ws.L_wide + s);         // known from the histogram of the whole input
            lbin = lkey >> 20;
          } else {
            // Fewer candidates than wished for (but at least k) and nothing known below the bound: lower it by
            // as much as would hold the missing ones at the density seen right above it -- what was never sent
            // piles up below the k-th, so half an octave down may hold a hundred times the wished-for number --
            // and by half an octave only where too few keys lie above the bound to tell.
            const uint32_t L_used = a.L_in[s], used = L_used >> 20;
            uint32_t pop = __ldcg(h + used), width = ((used + 1u) << 20) - L_used;
            if (pop < 64u && used + 1u < (uint32_t)kBins1) {
              pop += __ldcg(h + used + 1u);
              width += 1u << 20;
            }
            const float step = 1.5f * (float)(want + want / 16 - total) / (float)max(pop, 1u) * (float)width;
            if (pop >= 64u && step < (float)(4u << 20)) {
              const uint32_t down = (uint32_t)step + 1u;
              lkey = L_used > down ? L_used - down : 0u;
            } else {
              lkey = used > 4 ? (used - 4) << 20 : 0u;
            }
            lbin = lkey >> 20;
          }
          __syncthreads();
          // A bound of zero makes every element of the layer a candidate (zeros included).  That is fine for a
          // layer not much larger than the wished-for number of candidates; for a large one, no bound at all is
          // the better advice: the next selection finds nothing, notices, and takes its bound from a histogram.
          const uint32_t layer_cap = (ws.segs[s].tile_end - ws.segs[s].tile_begin) * (uint32_t)kWarpTile;
          const bool flood = lkey == 0 && layer_cap / 8 > want;
          if (threadIdx.x == 0) a.L_next[s] = flood ? 0xFFFFFFFFu : lkey;
        }
      }
      if (!everyone_picks) {   // the histogram has served; with one layer the others may still be reading it
        __syncthreads();
        for (int b = threadIdx.x; b < kBins1; b += kThreads) h[b] = 0;
      }
    }
    if (everyone_picks) {
      if (!failed || redo) break;
      // every CTA has seen the same histogram and comes here: clear it once all have read it, then redo
      if (!worker_barrier(ws.sync, Wb, ws.status, &sh.ok, bar_target, spin_limit)) return;
      if (cta == 0)
        for (int b = threadIdx.x; b < kBins1; b += kThreads) ws.hist1[b] = 0;
      if (!worker_barrier(ws.sync, Wb, ws.status, &sh.ok, bar_target, spin_limit)) return;
      redo = true;
    } else {
      if (!worker_barrier(ws.sync, Wb, ws.status, &sh.ok, bar_target, spin_limit)) return;
      if (redo || ld_volatile(ws.sync + kFail) == 0) break;
      redo = true;
    }
  }

  uint32_t near_seg = 0;   // layer of the candidate this thread looked at last (S > 1)
  // visits this thread's candidates in flat order: fn(value, index)
  auto each_own = [&](auto fn) {
    if (per_thread <= (uint32_t)kKeep) {
#pragma unroll
      for (int u = 0; u < kKeep; ++u)
        if (my_lo + u < my_hi) fn(rraw[u], ridx[u]);
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
            idx[u] = __ldcg(ws.cand_idx + cur.slot);
            cursor_advance(sh, parts, cur, 1);
          }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u)
          if (p + u < my_hi) fn(raw[u], idx[u]);
      }
    }
  };

  // ---- levels 2 and 3 ----------------------------------------------------------------
#pragma unroll 1
  for (int level = 2; level <= 3; ++level) {
    uint32_t* hist = level == 2 ? ws.hist2 : ws.hist3;
    constexpr int B = kBins2;   // both levels have 1024 bins
    const int SH = level == 2 ? 20 : 10;
    if (S == 1) {
      for (int b = threadIdx.x; b < B; b += kThreads) sh.stream.hist[b] = 0;
      __syncthreads();
      each_own([&](float v, uint32_t) {
        const uint32_t key = key_of(v);
        if ((key >> SH) == one_prefix) atomicAdd(sh.stream.hist + ((key >> (SH - 10)) & 1023u), 1u);
      });
      __syncthreads();
      for (int b = threadIdx.x; b < B; b += kThreads) {
        const uint32_t v = sh.stream.hist[b];
        if (v) atomicAdd(hist + b, v);
      }
      if (!worker_barrier(ws.sync, Wb, ws.status, &sh.ok, bar_target, spin_limit)) return;
      // the histogram of the level before has been read by everyone
      if (cta == 0) {
        uint32_t* old = level == 2 ? ws.hist1 : ws.hist2;
        for (int b = threadIdx.x; b < (level == 2 ? kBins1 : kBins2); b += kThreads) old[b] = 0;
      }
      uint32_t bin, krem;
      block_pick<B>(hist, one_krem, bin, krem, sh.warp_scan, sh.res);
      if (level == 2 && cta == 0 && one_wrem) {   // (CTA-uniform) the suggested bound: lower edge of the part that holds its entry
        uint32_t wsub, wleft;
        block_pick<B>(hist, one_wrem, wsub, wleft, sh.warp_scan, sh.res);
        if (threadIdx.x == 0) a.L_next[0] = ((one_prefix << 10) | wsub) << 10;
      }
      one_prefix = (one_prefix << 10) | bin;
      one_krem = krem;
    } else {
      if (seg_smem) {
        for (uint32_t s = threadIdx.x; s < S; s += kThreads) sm_seg_a[s] = __ldcg(&ws.sel[s].prefix);
        __syncthreads();
      }
      each_own([&](float v, uint32_t idx) {
        const uint32_t key = key_of(v);
        const uint32_t seg = seg_near(seg_off, S, idx, near_seg);
        const uint32_t prefix = seg_smem ? sm_seg_a[seg] : __ldcg(&ws.sel[seg].prefix);
        if ((key >> SH) == prefix) atomicAdd(hist + (size_t)seg * B + ((key >> (SH - 10)) & 1023u), 1u);
      });
      if (!worker_barrier(ws.sync, Wb, ws.status, &sh.ok, bar_target, spin_limit)) return;
      for (uint32_t s = cta; s < S; s += W) {
        uint32_t bin, krem;
        uint32_t* h = hist + (size_t)s * B;
        block_pick<B>(h, __ldcg(&ws.sel[s].krem), bin, krem, sh.warp_scan, sh.res);
        const uint32_t wrem = level == 2 ? __ldcg(&ws.sel[s].wrem) : 0u;   // written by this CTA at the first level
        if (wrem) {
          uint32_t wsub, wleft;
          block_pick<B>(h, wrem, wsub, wleft, sh.warp_scan, sh.res);
          if (threadIdx.x == 0) a.L_next[s] = ((__ldcg(&ws.sel[s].prefix) << 10) | wsub) << 10;
          __syncthreads();   // the prefix is read before it is extended below
        }
        if (threadIdx.x == 0) {
          const uint32_t pre = (__ldcg(&ws.sel[s].prefix) << 10) | bin;
          ws.sel[s].prefix = pre;
          ws.sel[s].krem = krem;
          if (level == 3) {
            ws.sel[s].T = pre;   // all 31 key bits are fixed now
            ws.sel[s].r = krem;
            ws.sel[s].neq = __ldcg(h + bin);
          }
        }
        __syncthreads();
        for (int b = threadIdx.x; b < B; b += kThreads) h[b] = 0;
      }
      if (!worker_barrier(ws.sync, Wb, ws.status, &sh.ok, bar_target, spin_limit)) return;
    }
  }

  // ---- count: (key > T, key == T) among this thread's candidates, prefix inside the CTA -------
  if (S > 1) {
    if (seg_smem) {
      for (uint32_t s = threadIdx.x; s < S; s += kThreads) {
        sm_seg_a[s] = __ldcg(&ws.sel[s].T);
        sm_seg_b[s] = __ldcg(&ws.sel[s].r);
      }
    }
    if (cta == 0) {
      // (key > T, key == T) candidates of all earlier layers: layer s selects k_s - r_s of the first kind
      unsigned long long carry = 0;
      for (uint32_t base = 0; base < S; base += kThreads) {
        const uint32_t s = base + threadIdx.x;
        unsigned long long v = 0;
        if (s < S) v = ((unsigned long long)(ws.segs[s].k[PM] - __ldcg(&ws.sel[s].r)) << 32) | __ldcg(&ws.sel[s].neq);
        unsigned long long total;
        const unsigned long long ex = block_excl_scan(v, sh.warp_scan, total) + carry;
        if (s < S) ws.seg_start[s] = make_uint2((uint32_t)(ex >> 32), (uint32_t)ex);
        carry += total;
      }
    }
    __syncthreads();
  }
  unsigned long long mine = 0;   // (gt << 32) | eq
  each_own([&](float v, uint32_t idx) {
    const uint32_t key = key_of(v);
    uint32_t T = one_prefix;
    if (S > 1) {
      const uint32_t seg = seg_near(seg_off, S, idx, near_seg);
      T = seg_smem ? sm_seg_a[seg] : __ldcg(&ws.sel[seg].T);
    }
    if (key > T) mine += 1ull << 32;
    else if (key == T) mine += 1ull;
  });
  unsigned long long cta_total;
  unsigned long long before = block_excl_scan(mine, sh.warp_scan, cta_total);
  if (threadIdx.x == 0) ws.cta_tot[cta] = make_uint2((uint32_t)(cta_total >> 32), (uint32_t)cta_total);
  if (!worker_barrier(ws.sync, Wb, ws.status, &sh.ok, bar_target, spin_limit)) return;
  if (S == 1 && cta == 0)
    for (int b = threadIdx.x; b < kBins3; b += kThreads) ws.hist3[b] = 0;

  // ---- emit: packet in index order, and the state updates that depend on selection ----
  {
    unsigned long long lower = 0;   // totals of the CTAs before this one (W <= kMaxWorkers)
    for (uint32_t c = threadIdx.x; c < cta; c += kThreads) {
      const uint2 q = __ldcg(ws.cta_tot + c);
      lower += ((unsigned long long)q.x << 32) | q.y;
    }
    unsigned long long lower_total;
    block_excl_scan(lower, sh.warp_scan, lower_total);
    before += lower_total;
    if (S > 1 && seg_smem) {
      for (uint32_t s = threadIdx.x; s < S; s += kThreads) sm_seg_start[s] = __ldcg(ws.seg_start + s);
      __syncthreads();
    }
    uint32_t gt_before = (uint32_t)(before >> 32), eq_before = (uint32_t)before;   // over all layers
    each_own([&](float val, uint32_t idx) {
      const uint32_t key = key_of(val);
      uint32_t T = one_prefix, r = one_krem, pkt_off = 0;
      uint2 start = make_uint2(0, 0);
      if (S > 1) {
        const uint32_t seg = seg_near(seg_off, S, idx, near_seg);
        T = seg_smem ? sm_seg_a[seg] : __ldcg(&ws.sel[seg].T);
        r = seg_smem ? sm_seg_b[seg] : __ldcg(&ws.sel[seg].r);
        start = seg_smem ? sm_seg_start[seg] : __ldcg(ws.seg_start + seg);
        pkt_off = ws.segs[seg].pkt_off[PM];
      }
      const bool is_gt = key > T, is_eq = key == T;
      const uint32_t eq_in_layer = eq_before - start.y;
      const bool sel = is_gt || (is_eq && eq_in_layer < r);
      if (sel) {
        const uint32_t pos = pkt_off + (gt_before - start.x) + min(eq_in_layer, r);
        const float q = round16(val, a.packet_format);   // what the packet carries (val itself with float32 packets)
        if (pos < a.pkt_count) {
          a.pkt_idx[pos] = idx;
          a.pkt_val[pos] = q;
        } else {
          atomicMin(ws.status, -1000 - MODE);
        }
        // Algorithm 1: the sent part leaves v (what a rounded packet did not carry stays: val - q, else zero).
        // Algorithm 3 keeps the sent entry's velocity t (already stored): no residual exists to take val - q.
        if (MODE == kPushResidual) out[idx] = __fsub_rn(val, q);
        if (MODE == kPull) {
          a.D[idx] = __fsub_rn(val, q);                  // Eq. 6b: v_k <- v_k + G; the rounding remainder stays
          if (a.theta_local) a.theta_local[idx] = __fadd_rn(a.theta_local[idx], q);  // Eq. 5
        }
      } else {
        if (MODE == kPushSam) out[idx] = __fmul_rn(val, a.inv_m);  // Eq. 12, lower branch
      }
      gt_before += is_gt ? 1u : 0u;
      eq_before += is_eq ? 1u : 0u;
    });
  }
  if (MODE == kPull && S == 1 && !redo && ws.plan != nullptr && ws.part_live != nullptr && cta == 0) {
    // Plan for the next pull's stream pass on this scratch set: its CTAs get ranges of tiles that cost
    // about the same, judged by what this pass cost each part (chunks read, candidates appended).  The
    // chunks that have to be read cluster in the tensors with the largest updates, and those tensors are
    // the same for every worker; with equal ranges a few CTAs do most of the reading.
    constexpr int PER = kMaxGrid / kThreads;
    const bool had = ld_volatile(ws.sync + kPlanParts) == parts && __ldcg(ws.plan + parts) == ws.num_tiles;
    uint32_t cost[PER], old_t0[PER];
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      const uint32_t p = j * kThreads + threadIdx.x;
      cost[j] = 0;
      old_t0[j] = 0;
      if (p < parts) {
        cost[j] = 4u + 8u * __ldcg(ws.part_live + p) + (sh.pre_cands[p + 1] - sh.pre_cands[p]) / 16u;
        old_t0[j] = had ? __ldcg(ws.plan + p) : part_first_tile(p, parts, ws.num_tiles);
      }
    }
    __syncthreads();   // pre_cands and slot0 have been read for the last time
    unsigned long long carry = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if ((uint32_t)(j * kThreads) < parts) {   // CTA-uniform
        const uint32_t p = j * kThreads + threadIdx.x;
        unsigned long long total;
        const unsigned long long ex = block_excl_scan(cost[j], sh.warp_scan, total) + carry;
        if (p < parts) {
          sh.pre_cands[p] = (uint32_t)ex;    // cost of the parts before p
          sh.slot0[p] = old_t0[j];
          sh.stream.hist[kMaxGrid + 1 + p] = cost[j];
        }
        carry += total;
      }
    }
    __syncthreads();
    const unsigned long long total_cost = carry;
    for (uint32_t j = threadIdx.x; j <= parts; j += kThreads) {
      uint32_t tile = j == 0 ? 0u : ws.num_tiles;
      if (j > 0 && j < parts) {
        const unsigned long long target = total_cost * j / parts;
        uint32_t lo = 0, hi = parts - 1;       // last part whose earlier parts cost no more than the target
        while (lo < hi) {
          const uint32_t mid = (lo + hi + 1) >> 1;
          if (sh.pre_cands[mid] <= target) lo = mid; else hi = mid - 1;
        }
        const uint32_t a0 = sh.slot0[lo], a1 = lo + 1 < parts ? sh.slot0[lo + 1] : ws.num_tiles;
        const unsigned long long into = target - sh.pre_cands[lo], c = sh.stream.hist[kMaxGrid + 1 + lo];
        tile = a0 + (uint32_t)((unsigned long long)(a1 - a0) * min(into, c) / c);
      }
      sh.stream.hist[j] = tile;
    }
    __syncthreads();
    // a part must not be longer than the pass can keep skip flags for; otherwise no plan
    int ok = 1;
    for (uint32_t j = threadIdx.x; j < parts; j += kThreads)
      if (sh.stream.hist[j + 1] < sh.stream.hist[j] || sh.stream.hist[j + 1] - sh.stream.hist[j] > 16384u) ok = 0;
    ok = __syncthreads_and(ok);
    for (uint32_t j = threadIdx.x; j < parts; j += kThreads) ws.plan[j] = sh.stream.hist[j];
    if (threadIdx.x == 0) {
      ws.plan[parts] = ok ? ws.num_tiles : 0u;
      ws.sync[kPlanParts] = parts;
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
// L_wide = a bound that admits about max(1.5 k, k+64) entries (the bound suggested for later selections)
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
    uint32_t wbin = 0, wrem = 0;
    const uint32_t want = spec_want(k);
    if (total >= want) block_pick<kBins1>(h, want, wbin, wrem, s_warp, s_res);
    if (threadIdx.x == 0) {
      ws.L_safe[s] = bin << 20;
      ws.L_wide[s] = total >= want ? bound_inside_bin(wbin, wrem, __ldcg(h + wbin), 0u) : 0u;
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

// ---- the pull's stream pass in its ring-less form (contexts with several workers) -----
__global__ void __maxnreg__(64) k_pull_light(Workspace ws, SelArgs a) {
  __shared__ StreamShared sh;
  if (blockIdx.x == 0 && threadIdx.x == 0) ws.sync[kBarCount] = 0;   // for the finalize launch that follows
  pull_tiles_light(ws, a, a.L_in, a.D, blockIdx.x, gridDim.x, sh);
}

// ---- pull without secondary compression: every nonzero entry of D_w -------------------
// The stream pass has run with the bound 1 for every layer (key >= 1 <=> the value is not zero),
// so the candidate buffer lists all nonzero entries of D_w in index order, part after part.
// This kernel copies the first `capacity` of them into the packet, clears them in D_w (Eq. 4:
// v_k becomes M), adds them to theta_w if kept (Eq. 5), and writes the count.
constexpr int kStatusLimit = -6;   // = DGS_ELIMIT
__global__ void __launch_bounds__(kThreads) k_emit_all(Workspace ws, float* __restrict__ D,
                                                       float* __restrict__ theta_local,
                                                       uint32_t* __restrict__ blk_max, uint32_t* __restrict__ out_idx,
                                                       float* __restrict__ out_val, uint32_t* __restrict__ out_count,
                                                       uint32_t capacity, int packet_format) {
  __shared__ uint32_t pre[kMaxGrid + 1], slot0[kMaxGrid];
  __shared__ unsigned long long warp_scan[kWarps];
  const uint32_t parts = ld_volatile(ws.sync + kParts);
  {
    constexpr int PER = kMaxGrid / kThreads;   // parts <= kMaxGrid
    unsigned long long carry = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if ((uint32_t)(j * kThreads) < parts) {   // CTA-uniform
        const uint32_t p = j * kThreads + threadIdx.x;
        const uint32_t cnt = p < parts ? __ldcg(ws.part_cands + p) : 0;
        if (p < parts) slot0[p] = __ldcg(ws.part_slot0 + p);
        unsigned long long total;
        const unsigned long long ex = block_excl_scan(cnt, warp_scan, total) + carry;
        if (p < parts) pre[p] = (uint32_t)ex;
        carry += total;
      }
    }
    if (threadIdx.x == 0) pre[parts] = (uint32_t)carry;
    __syncthreads();
  }
  const uint32_t C = pre[parts];
  const bool all = C <= capacity;          // every nonzero entry is sent: D_w is zero afterwards
  const uint32_t take = all ? C : capacity;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    *out_count = take;
    if (!all) atomicMin(ws.status, kStatusLimit);
    atomicAdd(ws.stats + 2, (unsigned long long)C);
  }
  for (uint32_t p = blockIdx.x * kThreads + threadIdx.x; p < take; p += gridDim.x * kThreads) {
    uint32_t lo = 0, hi = parts - 1;       // last part with pre[part] <= p
    while (lo < hi) {
      const uint32_t mid = (lo + hi + 1) >> 1;
      if (pre[mid] <= p) lo = mid; else hi = mid - 1;
    }
    const uint32_t slot = slot0[lo] + (p - pre[lo]);
    const uint32_t i = __ldcg(ws.cand_idx + slot);
    const float v = __ldcg(ws.cand_val + slot);
    const float q = round16(v, packet_format);
    out_idx[p] = i;
    out_val[p] = q;
    D[i] = __fsub_rn(v, q);      // zero with float32 packets; else what rounding left behind stays (Eq. 6b)
    if (theta_local != nullptr) theta_local[i] = __fadd_rn(theta_local[i], q);
    // the block's bound was made exact by the pass (a block without a nonzero entry already has bound 0);
    // with everything sent unrounded the whole block is zero now
    if (all && packet_format == 0 && blk_max != nullptr) blk_max[i / kWarpTile] = 0;
  }
  // the pass has added the candidates' top key bits to the layers' histograms: nobody reads them here
  const size_t words = (size_t)ws.num_segs * kBins1;
  for (size_t w = (size_t)blockIdx.x * kThreads + threadIdx.x; w < words; w += (size_t)gridDim.x * kThreads) ws.hist1[w] = 0;
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
constexpr int kCatchMaxPackets = 64;     // most packets one k_catch_up launch folds in
constexpr int kCatchCap = 1024;          // entries a CTA of k_catch_up can hold in shared memory (a power of two)
constexpr int kCatchSlots = 2 * kCatchCap;        // sparse pieces: slots of the table of distinct indices (>= 2 * kCatchCap)
constexpr int kCatchDense = 2 * kCatchSlots;      // dense pieces: elements of D a piece can mirror (= the bytes of the sparse table)
constexpr int kCatchLines = kCatchDense / 32;
constexpr uint32_t kCatchTarget = 3 * kCatchCap / 4;  // entries per range of the log the launch aims at (a range that holds more than kCatchCap is halved)
constexpr int kCatchMaxGrid = 16384;
constexpr int kCatchBlocks = kCatchCap / 8 < 16 ? 16 : kCatchCap / 8;   // blocks of D whose bounds a CTA of k_catch_up collects in shared memory first
constexpr int catch_log2(int v) { return v <= 1 ? 0 : 1 + catch_log2(v / 2); }
constexpr int kCatchSlotBits = catch_log2(kCatchSlots);
constexpr int kCatchThreads = 256;       // threads per CTA of k_catch_up (>= 2 * kCatchMaxPackets)

// Keeps a block's bound an upper bound on the magnitudes in the block.  Bounds only rise while
// packets are being subtracted, so a bound already read as high enough needs no atomic.
__device__ __forceinline__ void raise_bound(uint32_t* bound, uint32_t key) {
  if (key > __ldcg(bound)) atomicMax(bound, key);
}

struct PacketLog {
  uint32_t* idx;   // [ring][stride], each packet sorted by index
  float* val;      // [ring][stride]
  uint32_t stride; // entries between slots
  uint32_t cap;    // entries per packet
  uint32_t ring;   // slots
  // The index space is cut once, at the first packet filed, into `ranges` ranges that hold equally
  // many of that packet's entries (later packets are spread much alike): range g is
  // [bnd[g], bnd[g+1]), bnd[0] = 0, the last range is open-ended.  pos[slot][g] is the position of
  // the first entry of the packet in `slot` whose index is >= bnd[g]; pos[slot][ranges] = cap.
  uint32_t* bnd;   // [ranges]
  uint32_t* pos;   // [ring][ranges + 1]
  uint32_t ranges;
};

// The ranges of the log, from the quantiles of the first packet filed (sorted by index).
__global__ void __launch_bounds__(kThreads) k_log_ranges(const uint32_t* __restrict__ idx, PacketLog lg) {
  const uint32_t g = blockIdx.x * kThreads + threadIdx.x;
  if (g < lg.ranges) lg.bnd[g] = g == 0 ? 0u : idx[(uint64_t)g * lg.cap / lg.ranges];
}

// theta -= packet, and a copy of the packet into slot `slot` of the log: CTAs [0, copy_ctas).
// The remaining CTAs find where the ranges of the log begin in this packet.
__global__ void __launch_bounds__(kThreads) k_apply_log(const uint32_t* __restrict__ idx,
                                                        const float* __restrict__ val, uint32_t count,
                                                        float* __restrict__ theta, uint64_t n, int* status,
                                                        PacketLog lg, uint32_t slot, uint32_t copy_ctas) {
  if (blockIdx.x >= copy_ctas) {
    const uint32_t g = (blockIdx.x - copy_ctas) * kThreads + threadIdx.x;
    if (g > lg.ranges) return;
    uint32_t l = 0;
    if (g == lg.ranges) {
      l = count;
    } else if (g > 0) {
      const uint32_t key = __ldcg(lg.bnd + g);
      uint32_t r = count;
      while (l < r) {
        const uint32_t mid = (l + r) >> 1;
        if (__ldg(idx + mid) < key) l = mid + 1; else r = mid;
      }
    }
    lg.pos[(uint64_t)slot * (lg.ranges + 1) + g] = l;
    return;
  }
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

// D -= packets first .. first + count - 1 of the log, in that order (count <= kCatchMaxPackets).
// A CTA owns a range c of the log at a time; its part of every packet is known from the
// positions filed with the packet.  The values of D that the range's entries touch are brought
// into shared memory once, the packets' values are subtracted there in packet order (indices
// inside one packet are distinct, so a packet is one parallel step) and every value goes back
// once: every D[i] sees the same subtractions in the same order as if the packets had been
// applied one by one, with one trip to memory instead of one per packet.  No two CTAs touch the
// same entry of D.  A range with more entries than the tables hold (later packets much denser
// there than the one the ranges were taken from) is taken in several rounds, each over a piece
// of the range (halved until its entries fit).
//
// Two ways to hold a piece's values of D:
//   dense   the piece spans at most kCatchDense elements (counted from the 128-byte line its
//           first element lies in): shared memory mirrors the piece, an entry's place is its
//           offset.  Only the lines that hold an entry are read and written, each as one
//           coalesced 128-byte access of a warp, so the number of memory requests is the number
//           of lines touched, not the number of entries.  Where updates crowd -- the tensors
//           with the largest gradients, which take most entries of every packet -- a line holds
//           many entries.
//   sparse  a wider piece: a table of the distinct indices, one load and one store per index.
struct CatchShared {
  union {
    struct {
      uint32_t keys[kCatchSlots];        // sparse: index held by a slot, kFull = empty
      float vals[kCatchSlots];           //         running value of D at that index
    } tab;
    float dense[kCatchDense];            // dense: running values of D[a0 ..], a0 = first element of the piece's first line
  };
  uint16_t ent_slot[kCatchCap];          // place of each entry (packet-major order), 0xFFFF = index out of range
  float ent_val[kCatchCap];
  uint32_t lo[kCatchMaxPackets], hi[kCatchMaxPackets], end[kCatchMaxPackets];   // per packet: piece, end of the range
  uint32_t pre[kCatchMaxPackets + 1];    // exclusive prefix of hi - lo
  uint32_t bmax[kCatchBlocks];           // largest new magnitude per block of kWarpTile elements, from the piece's first block on
  uint32_t dirty[kCatchLines / 4];       // dense: one byte per line, nonzero = the line holds an entry
  uint32_t ab[2];                        // the range's first element and the element after its last
};
static_assert(sizeof(float) * kCatchDense == (sizeof(uint32_t) + sizeof(float)) * kCatchSlots, "the two views share their bytes");
static_assert(kCatchDense <= 0xFFFF && kCatchDense % kCatchThreads == 0 && kCatchThreads % 32 == 0 &&
              kCatchThreads >= 2 * kCatchMaxPackets, "offsets fit the entry table");
static_assert(kCatchDense / kWarpTile + 2 <= kCatchBlocks, "a dense piece's blocks fit the table of bounds");

__global__ void __maxnreg__(32) k_catch_up(PacketLog lg, uint64_t first, uint32_t count,
                                                       float* __restrict__ D, uint32_t* __restrict__ blk_max,
                                                       uint64_t n) {
  __shared__ __align__(16) CatchShared sh;
  const uint32_t tid = threadIdx.x;
  if (count == 0 || count > (uint32_t)kCatchMaxPackets) return;
  uint8_t* const dirty = reinterpret_cast<uint8_t*>(sh.dirty);
  // a CTA takes the ranges blockIdx.x, blockIdx.x + gridDim.x, ... one after the other; where a range lies
  // in the packets and in the index space is fetched one range ahead
  // (thread 2p reads where the range begins in packet p, thread 2p+1 where it ends)
  const uint32_t* const my_pos = lg.pos + ((first + (tid >> 1)) % lg.ring) * (uint64_t)(lg.ranges + 1) + (tid & 1u);
  uint32_t pos_ahead = 0, bnd_ahead = 0;     // of the range this CTA takes next
  if (blockIdx.x < lg.ranges) {
    if (tid < 2 * count) pos_ahead = __ldcg(my_pos + blockIdx.x);
    if (tid < 2) bnd_ahead = blockIdx.x + tid == 0 ? 0u : (blockIdx.x + tid == lg.ranges ? (uint32_t)n : __ldcg(lg.bnd + blockIdx.x + tid));
  }
  for (uint32_t c = blockIdx.x; c < lg.ranges; c += gridDim.x) {
  if (tid < 2 * count) {
    if (tid & 1u) sh.end[tid >> 1] = pos_ahead; else sh.lo[tid >> 1] = pos_ahead;
  }
  if (tid < 2) sh.ab[tid] = bnd_ahead;
  {
    const uint32_t cn = c + gridDim.x;
    if (cn < lg.ranges) {
      if (tid < 2 * count) pos_ahead = __ldcg(my_pos + cn);
      if (tid < 2) bnd_ahead = cn + tid == lg.ranges ? (uint32_t)n : __ldcg(lg.bnd + cn + tid);   // n < 2^32
    }
  }
  __syncthreads();
  const uint32_t range_b = sh.ab[1];
  uint32_t a = sh.ab[0];
  for (;;) {   // one round per piece [a, b) of the range; everything here is uniform over the CTA
    for (int s = tid; s < kCatchBlocks; s += kCatchThreads) sh.bmax[s] = 0;
    for (int s = tid; s < kCatchLines / 4; s += kCatchThreads) sh.dirty[s] = 0;   // (first written after the barriers below)
    // If what is left of the range fits a dense piece, its lines of D set out for shared memory now
    // (asynchronous 16-byte copies past L1), while the entries are being counted and gathered: where
    // updates crowd nearly every line holds an entry anyway, and a trip to memory leaves the chain.
    const bool ahead = range_b - (a & ~31u) <= (uint32_t)kCatchDense;
    if (ahead) {
      const uint32_t a0 = a & ~31u, floats = (range_b - a0 + 31u) & ~31u;   // whole lines; D is padded beyond n
      for (uint32_t q = tid * 4; q < floats; q += kCatchThreads * 4)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(sh.dense + q)), "l"(D + a0 + q) : "memory");
    }
    if (tid < count) sh.hi[tid] = sh.end[tid];
    uint32_t b = range_b;
    uint32_t E;
    for (;;) {
      __syncthreads();
      if (tid < 32) {
        // exclusive prefix of the pieces' lengths over the packets (two per lane)
        const uint32_t p0 = tid, p1 = tid + 32;
        const uint32_t x = p0 < count ? sh.hi[p0] - sh.lo[p0] : 0u, y = p1 < count ? sh.hi[p1] - sh.lo[p1] : 0u;
        uint32_t ix = x, iy = y;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const uint32_t ox = __shfl_up_sync(kFull, ix, d), oy = __shfl_up_sync(kFull, iy, d);
          if ((int)tid >= d) {
            ix += ox;
            iy += oy;
          }
        }
        const uint32_t tx = __shfl_sync(kFull, ix, 31), ty = __shfl_sync(kFull, iy, 31);
        if (p0 < count) sh.pre[p0] = ix - x;
        if (p1 < count) sh.pre[p1] = tx + iy - y;
        if (tid == 0) sh.pre[count] = tx + ty;
      }
      __syncthreads();
      E = sh.pre[count];
      if (E <= (uint32_t)kCatchCap || b - a <= 1) break;   // one index has at most `count` entries
      b = a + (b - a) / 2;
      if (tid < count) {
        const uint32_t* pi = lg.idx + ((first + tid) % lg.ring) * (uint64_t)lg.stride;
        uint32_t l = sh.lo[tid], r = sh.end[tid];
        while (l < r) {
          const uint32_t mid = (l + r) >> 1;
          if (__ldcg(pi + mid) < b) l = mid + 1; else r = mid;
        }
        sh.hi[tid] = l;
      }
    }
    if (E > 0 && E <= (uint32_t)kCatchCap) {
      const uint32_t a0 = a & ~31u;                         // first element of the line that holds a
      const uint32_t span = b - a0;                         // b <= n
      const bool dense = span <= (uint32_t)kCatchDense;
      if (!dense) {
        for (int s = tid; s < kCatchSlots; s += kCatchThreads) sh.tab.keys[s] = kFull;
        __syncthreads();
      }
      // gather: entry e (packet-major) -> its index and value; the index gets a place in shared memory
      constexpr int PER = kCatchCap / kCatchThreads;
      uint32_t ei[PER];
      float ev[PER];
#pragma unroll
      for (int u = 0; u < PER; ++u) {
        const uint32_t e = tid + u * kCatchThreads;
        ei[u] = kFull;
        ev[u] = 0.f;
        if (e < E) {
          uint32_t l = 0;                       // last packet p with pre[p] <= e: the same six probes for every
#pragma unroll                                  // entry, so that the searches of a thread's entries overlap
          for (uint32_t step = kCatchMaxPackets / 2; step >= 1; step >>= 1) {
            const uint32_t t = l + step;
            if (t < count && sh.pre[t] <= e) l = t;
          }
          const uint64_t at = ((first + l) % lg.ring) * (uint64_t)lg.stride + sh.lo[l] + (e - sh.pre[l]);
          ei[u] = __ldcg(lg.idx + at);
          ev[u] = __ldcg(lg.val + at);
        }
      }
#pragma unroll
      for (int u = 0; u < PER; ++u) {
        const uint32_t e = tid + u * kCatchThreads;
        if (e < E) {
          uint32_t slot = 0xFFFFu;
          const uint32_t i = ei[u];
          if (i < n && i >= a && i < b) {       // entries of a piece lie inside it; anything else is left alone
            if (dense) {
              slot = i - a0;
              dirty[slot >> 5] = 1;
            } else {
              uint32_t h = (i * 2654435761u) >> (32 - kCatchSlotBits);   // the top bits of the product
              for (;;) {
                const uint32_t old = atomicCAS(sh.tab.keys + h, kFull, i);
                if (old == kFull || old == i) break;
                h = (h + 1) & (kCatchSlots - 1);
              }
              slot = h;
            }
          }
          sh.ent_slot[e] = (uint16_t)slot;
          sh.ent_val[e] = ev[u];
        }
      }
      __syncthreads();
      float* const cur = dense ? sh.dense : sh.tab.vals;    // running values, by place
      constexpr int SPT = kCatchSlots / kCatchThreads;      // sparse: table slots per thread
      constexpr int EPT = kCatchDense / kCatchThreads;      // dense: elements per thread, element tid + j * kCatchThreads
      constexpr int LB = EPT < 8 ? EPT : 8;                  // loads a thread has in flight together
      if (dense && ahead) {
        asm volatile("cp.async.wait_all;" ::: "memory");   // the lines that set out at the start of the piece
      } else if (dense) {
        // a warp's 32 threads hold one line at every step j: one 128-byte request per line that holds an entry
#pragma unroll 1
        for (int j0 = 0; j0 < EPT; j0 += LB) {
          if ((uint32_t)(j0 * kCatchThreads) >= span) break;
          float d[LB];
#pragma unroll
          for (int j = 0; j < LB; ++j) {
            const uint32_t off = tid + (j0 + j) * kCatchThreads;
            d[j] = 0.f;
            if (off < span && dirty[off >> 5]) d[j] = __ldcg(D + a0 + off);
          }
#pragma unroll
          for (int j = 0; j < LB; ++j) sh.dense[tid + (j0 + j) * kCatchThreads] = d[j];
        }
      } else {
        // one load of D per distinct index, all in flight together
        uint32_t k[SPT];
        float d[SPT];
#pragma unroll
        for (int u = 0; u < SPT; ++u) {
          k[u] = sh.tab.keys[tid + u * kCatchThreads];
          d[u] = 0.f;
          if (k[u] != kFull) d[u] = __ldcg(D + k[u]);
        }
#pragma unroll
        for (int u = 0; u < SPT; ++u)
          if (k[u] != kFull) sh.tab.vals[tid + u * kCatchThreads] = d[u];
      }
      __syncthreads();
      // The packets in arrival order; inside one packet every index, and so every place, occurs once, so a
      // packet's part is one parallel step.  A part of a piece rarely has more entries than a warp has lanes:
      // one warp takes the steps one after the other with only its own barrier between them, which costs a
      // fraction of a barrier of the whole CTA per packet.
      if (tid < 32) {
        constexpr int G = 4;   // packets whose entries a lane fetches together, ahead of the steps that use them
        for (uint32_t p0 = 0; p0 < count; p0 += G) {
          uint32_t slot[G], e1[G];
          float val[G];
          uint32_t ebeg = sh.pre[p0];
#pragma unroll
          for (int j = 0; j < G; ++j) {
            const uint32_t pend = p0 + j < count ? sh.pre[p0 + j + 1] : ebeg;
            const uint32_t e = ebeg + tid;
            slot[j] = 0xFFFFu;
            val[j] = 0.f;
            if (e < pend) {
              slot[j] = sh.ent_slot[e];
              val[j] = sh.ent_val[e];
            }
            e1[j] = pend;
            ebeg = pend;
          }
          ebeg = sh.pre[p0];
#pragma unroll
          for (int j = 0; j < G; ++j) {
            if (slot[j] != 0xFFFFu) cur[slot[j]] = __fsub_rn(cur[slot[j]], val[j]);
            for (uint32_t e = ebeg + 32 + tid; e < e1[j]; e += 32) {   // a part with more entries than lanes
              const uint32_t sl = sh.ent_slot[e];
              if (sl != 0xFFFFu) cur[sl] = __fsub_rn(cur[sl], sh.ent_val[e]);
            }
            __syncwarp();
            ebeg = e1[j];
          }
        }
      }
      __syncthreads();
      // Back to memory.  The blocks' bounds must stay upper bounds: the largest new magnitude per block is
      // collected in shared memory, one global atomic per block afterwards.
      if (dense) {
        // A warp takes four consecutive lines at a time (their dirty flags are one word); the loads of the
        // four are in flight together, and a block's bound gets one reduction where the four lie in one block.
        const uint32_t lead = a - a0;            // elements of the first line that belong to the range before
        const uint32_t blk0 = a / kWarpTile, line0 = a0 >> 5;
        const uint32_t lines = (span + 31u) >> 5, lane = tid & 31u;
#pragma unroll 1
        for (uint32_t l0 = (tid >> 5) * 4; l0 < lines; l0 += (kCatchThreads / 32) * 4) {
          const uint32_t flags = sh.dirty[l0 >> 2];
          if (flags == 0) continue;
          uint32_t key[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const uint32_t off = (l0 + u) * 32 + lane;
            key[u] = 0;
            if (((flags >> (8 * u)) & 0xFFu) && off < span && off >= lead) {
              const float r = sh.dense[off];
              __stcg(D + a0 + off, r);
              key[u] = key_of(r);
            }
          }
          // a line lies inside one block (lines and blocks start at multiples of 32 and of kWarpTile)
          const uint32_t b_first = (line0 + l0) / (kWarpTile / 32) - blk0, b_last = (line0 + l0 + 3) / (kWarpTile / 32) - blk0;
          if (b_first == b_last) {
            const uint32_t k4 = __reduce_max_sync(kFull, max(max(key[0], key[1]), max(key[2], key[3])));
            if (lane == 0 && k4) atomicMax(sh.bmax + b_first, k4);
          } else {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const uint32_t k1 = __reduce_max_sync(kFull, key[u]);
              if (lane == 0 && k1) atomicMax(sh.bmax + ((line0 + l0 + u) / (kWarpTile / 32) - blk0), k1);
            }
          }
        }
      } else {
#pragma unroll
        for (int u = 0; u < SPT; ++u) {
          const uint32_t i = sh.tab.keys[tid + u * kCatchThreads];
          if (i != kFull) {
            const float r = sh.tab.vals[tid + u * kCatchThreads];
            __stcg(D + i, r);
            const uint32_t blk = i / kWarpTile - a / kWarpTile;
            if (blk < (uint32_t)kCatchBlocks) atomicMax(sh.bmax + blk, key_of(r));
            else atomicMax(blk_max + i / kWarpTile, key_of(r));   // a piece spanning more blocks than the table holds
          }
        }
      }
      __syncthreads();
      for (int s = tid; s < kCatchBlocks; s += kCatchThreads) {
        const uint32_t v = sh.bmax[s];
        if (v) atomicMax(blk_max + a / kWarpTile + s, v);
      }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");   // (copies of a piece that turned out empty: nothing may still land)
    if (b == range_b) break;
    __syncthreads();   // the tables and the pieces are read until here
    if (tid < count) sh.lo[tid] = sh.hi[tid];
    a = b;
  }
  __syncthreads();   // the tables are free for the next range
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
  if (q < num_workers) raise_bound(blk_max + (uint64_t)q * blk_stride + i / kWarpTile, key_of(r));
}

}  // namespace dgs
