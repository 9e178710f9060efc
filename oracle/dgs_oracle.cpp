// CPU checker for the DGS push / apply / pull loop (arXiv 1910.10929).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
// method computes, used to judge the CUDA library.  Nothing in the product path
// may call it; it shares no code with the CUDA sources and is built on its own
// (g++ -O2 -ffp-contract=off, no fast-math, single thread).
//
// Every floating-point step below is ONE correctly rounded IEEE binary32
// operation in the order written, so a GPU implementation that uses the same
// operations in the same order must agree bit for bit.
//
// State kept (all float32):
//   theta[n]          global model, theta_t = theta_0 + M_t               (Eq. 2)
//   u[N][n]           per-worker SAMomentum velocity, starts at 0         (Algorithm 3, init)
//   D[N][n]           per-worker model difference  D_k = M - v_k, starts 0 (Eq. 3; Algorithm 2, init)
//   theta_local[N][n] optional worker copies, start at theta_0            (Algorithm 3, init; Eq. 5)
//
// Readings taken where the paper leaves a choice:
//   * "thr <- R% of |x|" + "Mask <- |x| > thr" is read as: keep EXACTLY k entries
//     per layer, ordered by (|x| descending, index ascending); |x| compared
//     through its bit pattern with the sign cleared, so +0 and -0 tie.
//   * the server's per-worker vector moves by v_k <- v_k + G (Eq. 4, Eq. 6b); the
//     minus sign in the last-but-one line of Algorithm 2 contradicts both.
//   * D_k is stored instead of (M, v_k): M - decode(g) lowers every D_k by the
//     packet, and v_k <- v_k + G lowers D_k by G, i.e. clears the sent entries.
//   * unsent velocity entries are multiplied once by fl(1/m)  (Eq. 12 form).
//   * a pull without secondary compression sends every entry of D_k that is not zero
//     (+0 and -0 both count as zero) and clears it.
//   * with 16-bit packet values (not in the paper's algorithms; its closing section names the
//     direction): selection by the unrounded magnitudes; the packet carries q = round16(value); a
//     push leaves the worker's velocity as Eq. 12 says (no residual exists to take t - q); a pull
//     lowers D_k by q, so that what rounding left behind stays with the server (Eq. 6b).
//
// parity pins: see tests/test_oracle_*.py (brute-force sort, hand-worked example,
// dense limit = serial momentum ASGD, Eq. 13 telescoping, Eq. 12, exact split).
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <functional>
#include <vector>

namespace {

inline uint32_t key_of(float x) {          // |x| as an unsigned integer, monotone in |x|
  uint32_t b;
  std::memcpy(&b, &x, 4);
  return b & 0x7FFFFFFFu;
}

// Packet values in a 16-bit floating-point format (the paper's closing section proposes combining the
// method with other compression; here: the VALUES of a packet are rounded, the selection is untouched).
// fmt 0: none.  fmt 1: bfloat16 (8 exponent bits, 7 fraction bits).  fmt 2: IEEE binary16 (5 exponent
// bits, 10 fraction bits, gradual underflow); magnitudes that would round beyond the largest finite
// binary16 number, 65504, are sent as 65504 (no infinities in a packet).  Round to nearest, ties to even.
// The result is returned as the float32 number with that value.  Inputs are finite.
float round16(float x, int fmt) {
  uint32_t b;
  std::memcpy(&b, &x, 4);
  const uint32_t sign = b & 0x80000000u;
  uint32_t m = b & 0x7FFFFFFFu;            // bits of |x|
  if (fmt == 1) {
    m += 0x7FFFu + ((m >> 16) & 1u);       // nearest multiple of 2^16 in the bit pattern, ties to even
    m &= 0xFFFF0000u;
    if (m >= 0x7F800000u) m = 0x7F7F0000u; // would be infinite: largest finite bfloat16
  } else if (fmt == 2) {
    if (m >= 0x477FF000u) {                // |x| >= 65520 = the midpoint above 65504: saturate
      m = 0x477FE000u;                     // 65504
    } else if (m >= 0x38800000u) {         // |x| >= 2^-14: a normal binary16, 13 fraction bits are dropped
      m += 0xFFFu + ((m >> 13) & 1u);
      m &= 0xFFFFE000u;
    } else {
      // below 2^-14 binary16 steps by 2^-24: |x| / 2^-24 rounded to an integer (exact scaling by a power of two)
      float ax;
      std::memcpy(&ax, &m, 4);
      const float scaled = ax * 16777216.0f;               // exact: < 2^10
      float r = static_cast<float>(static_cast<int>(scaled));
      const float frac = scaled - r;                         // exact
      if (frac > 0.5f || (frac == 0.5f && (static_cast<int>(r) & 1))) r += 1.0f;
      const float back = r * (1.0f / 16777216.0f);           // exact
      std::memcpy(&m, &back, 4);
    }
  } else {
    return x;
  }
  m |= sign;
  float y;
  std::memcpy(&y, &m, 4);
  return y;
}

// TOPK(x, k): order by (key descending, index ascending), take the first k.
// Returns the chosen positions in ascending order.
void topk(const float* x, uint64_t len, uint64_t k, std::vector<uint64_t>& chosen) {
  chosen.clear();
  if (k == 0) return;
  std::vector<uint32_t> keys(len);
  for (uint64_t i = 0; i < len; ++i) keys[i] = key_of(x[i]);
  std::vector<uint32_t> work(keys);
  std::nth_element(work.begin(), work.begin() + (k - 1), work.end(), std::greater<uint32_t>());
  const uint32_t T = work[k - 1];          // k-th largest key
  uint64_t above = 0;
  for (uint64_t i = 0; i < len; ++i) above += keys[i] > T;
  uint64_t ties_left = k - above;          // how many entries equal to T still fit
  for (uint64_t i = 0; i < len; ++i) {
    if (keys[i] > T) {
      chosen.push_back(i);
    } else if (keys[i] == T && ties_left > 0) {
      chosen.push_back(i);
      --ties_left;
    }
  }
}

struct Oracle {
  uint64_t n = 0;
  uint32_t N = 0, S = 0;
  float lr = 0, m = 0, inv_m = 0;
  int keep_local = 0;
  int residual_mode = 0;                   // 1: Algorithm 1 (plain residual, no momentum)
  int packet_format = 0;                   // 0: float32 values; 1: bfloat16; 2: binary16 (see round16)
  std::vector<uint64_t> off, len;
  std::vector<uint32_t> k_push, k_pull;
  std::vector<float> theta;
  std::vector<std::vector<float>> u, D, theta_local;
  std::vector<float> t;                    // scratch: the pre-selection velocity of one push
  uint64_t stamp = 0;                      // server timestamp t
  std::vector<int64_t> prev;               // prev(k)
};

}  // namespace

extern "C" {

// The rounding of packet values, on its own (for pinning it).
float dgs_oracle_round16(float x, int fmt) { return round16(x, fmt); }

// Standalone selection, for pinning TOPK by brute force. out_pos receives k ascending positions.
void dgs_oracle_topk(const float* x, uint64_t len, uint64_t k, uint64_t* out_pos) {
  std::vector<uint64_t> c;
  topk(x, len, k, c);
  for (uint64_t j = 0; j < c.size(); ++j) out_pos[j] = c[j];
}

void* dgs_oracle_create(uint64_t n, uint32_t N, float lr, float m, uint32_t S,
                        const uint64_t* seg_off, const uint64_t* seg_len,
                        const uint32_t* k_push, const uint32_t* k_pull,
                        const float* theta0, int keep_local, int residual_mode, int packet_format) {
  Oracle* o = new Oracle;
  o->packet_format = packet_format;
  o->n = n; o->N = N; o->S = S; o->lr = lr; o->m = m;
  o->inv_m = 1.0f / m;                     // one IEEE division, then used as a constant
  o->keep_local = keep_local;
  o->residual_mode = residual_mode;
  o->off.assign(seg_off, seg_off + S);
  o->len.assign(seg_len, seg_len + S);
  o->k_push.assign(k_push, k_push + S);
  o->k_pull.assign(k_pull, k_pull + S);
  o->theta.assign(theta0, theta0 + n);
  o->u.assign(N, std::vector<float>(n, 0.0f));
  o->D.assign(N, std::vector<float>(n, 0.0f));
  if (keep_local) o->theta_local.assign(N, std::vector<float>(theta0, theta0 + n));
  o->t.assign(n, 0.0f);
  o->prev.assign(N, -1);
  return o;
}

void dgs_oracle_free(void* h) { delete static_cast<Oracle*>(h); }

// Worker push (Algorithm 3, the velocity update through encode()).
// Writes sum(k_push) (index, value) pairs, ascending index. Returns the count.
uint64_t dgs_oracle_push(void* h, uint32_t w, const float* grad, uint32_t* out_idx, float* out_val) {
  Oracle& o = *static_cast<Oracle*>(h);
  std::vector<float>& u = o.u[w];
  float* t = o.t.data();
  if (!o.residual_mode) {
    // u <- m*u + eta*grad : two products, one sum, each rounded (no fused multiply-add)
    for (uint64_t i = 0; i < o.n; ++i) {
      const float a = o.m * u[i];
      const float b = o.lr * grad[i];
      t[i] = a + b;
    }
  } else {
    // Algorithm 1: v <- v + eta*grad
    for (uint64_t i = 0; i < o.n; ++i) {
      const float b = o.lr * grad[i];
      t[i] = u[i] + b;
    }
  }
  uint64_t cnt = 0;
  std::vector<uint64_t> chosen;
  for (uint32_t s = 0; s < o.S; ++s) {      // per-layer loop
    const uint64_t base = o.off[s], L = o.len[s];
    topk(t + base, L, o.k_push[s], chosen);
    // default: every entry is "unsent"
    if (!o.residual_mode) {
      for (uint64_t i = 0; i < L; ++i) u[base + i] = t[base + i] * o.inv_m;   // Eq. 12, lower branch
    } else {
      for (uint64_t i = 0; i < L; ++i) u[base + i] = t[base + i];             // residual kept
    }
    for (uint64_t p : chosen) {             // sent entries
      const uint64_t i = base + p;
      const float q = round16(t[i], o.packet_format);   // what the packet carries
      out_idx[cnt] = static_cast<uint32_t>(i);
      out_val[cnt] = q;
      ++cnt;
      // Eq. 12 upper branch: the velocity of a sent entry stays t (SAMomentum keeps no residual, so the
      // rounding of a packet value is not fed back).  Algorithm 1: the sent part leaves the residual,
      // which keeps what the packet did not carry (t - q; zero without rounding).
      u[i] = o.residual_mode ? t[i] - q : t[i];
    }
  }
  return cnt;
}

// Server apply (Algorithm 2: M <- M - decode(g); every D_k = M - v_k moves with M).
void dgs_oracle_apply(void* h, uint32_t /*w*/, const uint32_t* idx, const float* val, uint64_t count) {
  Oracle& o = *static_cast<Oracle*>(h);
  for (uint64_t j = 0; j < count; ++j) {
    const uint64_t i = idx[j];
    o.theta[i] = o.theta[i] - val[j];
    for (uint32_t q = 0; q < o.N; ++q) o.D[q][i] = o.D[q][i] - val[j];
  }
  o.stamp += 1;
}

// Worker pull with secondary compression (Eq. 6a, 6b; Algorithm 2's per-layer loop; Eq. 5).
uint64_t dgs_oracle_pull(void* h, uint32_t w, uint32_t* out_idx, float* out_val) {
  Oracle& o = *static_cast<Oracle*>(h);
  std::vector<float>& D = o.D[w];
  uint64_t cnt = 0;
  std::vector<uint64_t> chosen;
  for (uint32_t s = 0; s < o.S; ++s) {
    const uint64_t base = o.off[s];
    topk(D.data() + base, o.len[s], o.k_pull[s], chosen);
    for (uint64_t p : chosen) {
      const uint64_t i = base + p;
      const float q = round16(D[i], o.packet_format);                       // what the packet carries
      out_idx[cnt] = static_cast<uint32_t>(i);
      out_val[cnt] = q;
      ++cnt;
      if (o.keep_local) o.theta_local[w][i] = o.theta_local[w][i] + q;      // Eq. 5
      D[i] = D[i] - q;                            // v_k <- v_k + G (Eq. 6b): zero, or what rounding left behind
    }
  }
  o.prev[w] = static_cast<int64_t>(o.stamp);
  return cnt;
}

// Worker pull WITHOUT secondary compression (Algorithm 2 with the switch off; the paper's normal
// case: "there is no secondary compression for G"): the server sends all of G_k = M - v_k, which is
// sparse, and v_k becomes M (Eq. 3, Eq. 4).  In accumulator form: every nonzero entry of D_k is
// sent, in ascending index order, and cleared, so that D_k is zero afterwards; the worker adds G
// to its model (Eq. 5).  At most `cap` entries are written; returns how many D_k held (the caller
// sees an overflow as a return value above cap; entries beyond cap are neither sent nor cleared).
uint64_t dgs_oracle_pull_all(void* h, uint32_t w, uint32_t* out_idx, float* out_val, uint64_t cap) {
  Oracle& o = *static_cast<Oracle*>(h);
  std::vector<float>& D = o.D[w];
  uint64_t cnt = 0;
  for (uint64_t i = 0; i < o.n; ++i) {
    if (D[i] != 0.0f) {
      if (cnt < cap) {
        const float q = round16(D[i], o.packet_format);
        out_idx[cnt] = static_cast<uint32_t>(i);
        out_val[cnt] = q;
        if (o.keep_local) o.theta_local[w][i] = o.theta_local[w][i] + q;      // Eq. 5
        D[i] = D[i] - q;                          // v_k <- v_k + G = M (Eq. 4), up to what rounding left behind
      }
      ++cnt;
    }
  }
  o.prev[w] = static_cast<int64_t>(o.stamp);
  return cnt;
}

// which: 0 theta, 1 u[w], 2 D[w], 3 theta_local[w]
const float* dgs_oracle_state(void* h, int which, uint32_t w) {
  Oracle& o = *static_cast<Oracle*>(h);
  switch (which) {
    case 0: return o.theta.data();
    case 1: return o.u[w].data();
    case 2: return o.D[w].data();
    case 3: return o.keep_local ? o.theta_local[w].data() : nullptr;
  }
  return nullptr;
}

uint64_t dgs_oracle_timestamp(void* h) { return static_cast<Oracle*>(h)->stamp; }
int64_t dgs_oracle_prev(void* h, uint32_t w) { return static_cast<Oracle*>(h)->prev[w]; }

}  // extern "C"
