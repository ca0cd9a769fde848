// CPU oracle for the routed mixture-of-experts layer with FP4 expert weights.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
// tests, the smoke check and the benchmark's cpu_baseline leg compare the CUDA
// library against.  It shares no code, header, table or helper with the CUDA
// path and nothing on the product path may call it.
//
// What it restates (paper, "Execution structure" figure and the accepted
// large-prefill path in "Prefill optimization"): Router Top-k -> route
// production (expert sorter) -> FP4 routed experts gate/up -> activation
// rounded to BF16 -> down projection with FP32 per-slot partials stored to
// unique slots -> fixed-order Top-k FP32 reduction.  The paper gives the layer
// in prose only; every point it leaves open is fixed by the readings listed in
// the repository's design notes (G1..G14) and repeated beside the code here.
//
// Precision: the workload statement fixes fp32 accumulation, so the primary
// entry points accumulate in fp32 in ascending index order.  `acc64 != 0`
// selects a twin that accumulates the two contractions in fp64 (used as a pin
// on the fp32 one, never as the expected value of a GPU test).
//
// Build: g++ -O2 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
// (no implicit fused multiply-add: only the explicit std::fmaf calls fuse).
//
// Pins (tests/test_oracle_*.py): the printed E2M1 magnitude list, 2^(b-127),
// exp() in double, a full sort, numpy stable argsort, the printed block
// permutation and its inverse, a dense SwiGLU MLP in float64, brute-force
// dense evaluation of every expert, exact-scaling and single-weight cases, and
// an exact-rational fmaf recurrence.  No function here is "parity unpinned".

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---- scalar formats -------------------------------------------------------

// E2M1 (4-bit float): bit 3 sign, bits 2:1 exponent with bias 1, bit 0
// mantissa.  Exponent 0 is the subnormal binade {0, 0.5}.  The paper lists the
// doubled magnitudes 0,1,2,3,4,6,8,12 (historical TP4/EP1 decode route).
inline float e2m1_value(unsigned code) {
  const unsigned s = (code >> 3) & 1u, e = (code >> 1) & 3u, m = code & 1u;
  const float mag = (e == 0u) ? 0.5f * static_cast<float>(m)
                              : std::ldexp(1.0f + 0.5f * static_cast<float>(m), static_cast<int>(e) - 1);
  return s ? -mag : mag;
}

// E8M0 block scale: byte b means 2^(b-127); 255 is NaN (reading G9).
inline float e8m0_value(unsigned b) {
  if (b == 255u) return std::nanf("");
  return std::ldexp(1.0f, static_cast<int>(b) - 127);
}

inline float bf16_to_f32(uint16_t h) {
  uint32_t u = static_cast<uint32_t>(h) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

// round-to-nearest-even fp32 -> bf16
inline uint16_t f32_to_bf16(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<uint16_t>((u >> 16) | 0x0040u);  // NaN stays NaN
  const uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return static_cast<uint16_t>(u >> 16);
}

// The specified exponential of the routing softmax (reading G2).  The routing
// weights must be bit-identical on CPU and GPU, so the exponential is a fixed
// sequence of fp32 operations instead of a library call:
//   d  <- max(d, -80)
//   n  = rint(d * log2e)                      (ties to even)
//   r  = fma(n, -ln2_hi, d); r = fma(n, -ln2_lo, r)
//   p  = 1 + r + r^2/2 + ... + r^6/720        (Horner, every step an fma)
//   EXP(d) = p * 2^n                          (exact: result stays normal)
inline float exp_spec(float d) {
  if (d < -80.0f) d = -80.0f;
  const float t = d * 1.44269504f;
  const float n = std::rint(t);
  float r = std::fmaf(n, -0.693145752f, d);
  r = std::fmaf(n, -1.42860677e-6f, r);
  float p = 1.0f / 720.0f;
  p = std::fmaf(p, r, 1.0f / 120.0f);
  p = std::fmaf(p, r, 1.0f / 24.0f);
  p = std::fmaf(p, r, 1.0f / 6.0f);
  p = std::fmaf(p, r, 0.5f);
  p = std::fmaf(p, r, 1.0f);
  p = std::fmaf(p, r, 1.0f);
  return std::ldexp(p, static_cast<int>(n));
}

// The two decodes above, tabulated once (16 and 256 entries) so the inner loops
// below do not call ldexp per weight; the tables hold exactly the values the
// functions return.
struct DecodeTables {
  float e2m1[16];
  float e8m0[256];
  DecodeTables() {
    for (unsigned c = 0; c < 16; ++c) e2m1[c] = e2m1_value(c);
    for (unsigned b = 0; b < 256; ++b) e8m0[b] = e8m0_value(b);
  }
};
const DecodeTables& tables() {
  static const DecodeTables t;
  return t;
}

// weight value of element (row, h) of one expert matrix [rows, K] stored as
// packed codes [rows, K/2] (element 2j in bits 3:0 of byte j, element 2j+1 in
// bits 7:4; reading G3) with one scale byte per (row, 32 consecutive K):
// value = E2M1(code) * 2^(scale_byte - 127)  (exact: a power-of-two scaling).
inline float weight_value(const uint8_t* codes, const uint8_t* scales, int64_t K, int64_t row, int64_t h) {
  const DecodeTables& t = tables();
  const uint8_t byte = codes[row * (K / 2) + h / 2];
  const unsigned code = (h & 1) ? (byte >> 4) : (byte & 0xFu);
  return t.e2m1[code] * t.e8m0[scales[row * (K / 32) + h / 32]];
}

// ---- routing for one token -------------------------------------------------

// Top-k by raw logit, slot 0 the largest, equal logits -> lower expert id
// (readings G1, G7); weights = softmax over the k selected logits using
// exp_spec, summed left to right in fp32, IEEE division.
void route_token(const float* l, int E, int k, int32_t* ids, float* w) {
  std::vector<char> taken(static_cast<size_t>(E), 0);
  for (int j = 0; j < k; ++j) {
    int best = -1;
    for (int e = 0; e < E; ++e) {
      if (taken[e]) continue;
      if (best < 0 || l[e] > l[best]) best = e;  // strict '>' : first (lowest id) of equals wins
    }
    taken[best] = 1;
    ids[j] = best;
  }
  const float m = l[ids[0]];
  std::vector<float> ex(static_cast<size_t>(k));
  float s = 0.0f;
  for (int j = 0; j < k; ++j) {
    ex[j] = exp_spec(l[ids[j]] - m);
    s = (j == 0) ? ex[0] : s + ex[j];
  }
  for (int j = 0; j < k; ++j) w[j] = ex[j] / s;
}

// ---- online activation quantisation (variant) --------------------------------
//
// The paper's historical decode route quantises the BF16 activations online to INT8, one scale per 32 elements,
// so that an integer dot product can consume them.  The analogue on the hardware this repository targets is the
// weights' own format: E2M1 codes with one E8M0 scale byte per 32 consecutive elements (reading G18).  One block:
//   amax = max |v|;  amax = 0 -> byte 127, every code a signed zero;
//   s    = the smallest integer in [-126, 126] with amax <= 6 * 2^s  (6 = largest E2M1 magnitude: nothing saturates,
//          and a smaller s would);  scale byte = s + 127;
//   code = sign bit of v, magnitude = the E2M1 magnitude nearest to |v| / 2^s, a tie going to the magnitude whose
//          mantissa bit is 0 (round to nearest even); dequantised value = E2M1(code) * 2^s.
// |v| / 2^s is formed in double, where it is exact for every bf16 v.  Domain: |v| <= 2^126, so that every decoded
// value is an fp32 number (above it 4 * 2^126 or 6 * 2^126 would not be); activations never come near it.
inline void quant_block(const float* v, uint8_t* codes /* 32, one per byte */, uint8_t* scale_byte) {
  double amax = 0.0;
  for (int j = 0; j < 32; ++j) amax = std::fmax(amax, std::fabs(static_cast<double>(v[j])));
  int s = 0;
  if (amax > 0.0) {
    s = -126;
    while (s < 126 && amax > 6.0 * std::ldexp(1.0, s)) s += 1;
  }
  *scale_byte = static_cast<uint8_t>(s + 127);
  for (int j = 0; j < 32; ++j) {
    const double m = std::fabs(static_cast<double>(v[j])) / std::ldexp(1.0, s);
    unsigned best = 0;
    double best_d = m;  // distance to magnitude code 0 (value 0)
    for (unsigned c = 1; c < 8; ++c) {
      const double d = std::fabs(m - static_cast<double>(e2m1_value(c)));
      if (d < best_d || (d == best_d && (c & 1u) == 0u)) {
        best = c;
        best_d = d;
      }
    }
    codes[j] = static_cast<uint8_t>(best | (std::signbit(v[j]) ? 8u : 0u));
  }
}

// A row of K bf16 values -> the values its quantised form decodes to (what the contraction then consumes), and
// optionally the packed codes (element 2j in the low nibble of byte j, as the weights) and scale bytes.
inline void quant_row(const uint16_t* row, int64_t K, float* deq, uint8_t* packed /* K/2 or NULL */,
                      uint8_t* scales /* K/32 or NULL */) {
  for (int64_t b = 0; b < K / 32; ++b) {
    float v[32];
    uint8_t codes[32], sb;
    for (int j = 0; j < 32; ++j) v[j] = bf16_to_f32(row[b * 32 + j]);
    quant_block(v, codes, &sb);
    for (int j = 0; j < 32; ++j) deq[b * 32 + j] = e2m1_value(codes[j]) * e8m0_value(sb);
    if (packed != nullptr)
      for (int j = 0; j < 16; ++j) packed[b * 16 + j] = static_cast<uint8_t>(codes[2 * j] | (codes[2 * j + 1] << 4));
    if (scales != nullptr) scales[b] = sb;
  }
}

// ---- one slot of the expert FFN ---------------------------------------------

// act[i] = bf16( silu(g_i) * u_i ), g = W1 x, u = W3 x, W1 = rows [0,I) of w13,
// W3 = rows [I,2I) (reading G4); g and u are not rounded before the
// activation (reading G6); y[n] = sum_i W2[n,i] act[i].  Accumulation in
// ascending index order in ACC (float or double).
//
// quant = true is the quantised-activation variant: both contractions consume the quantised form of their input row
// (quant_row: the token row; the intermediate after its rounding to bf16), everything else unchanged.
template <typename ACC>
void ffn_slot(const uint16_t* x_row, const uint8_t* w13, const uint8_t* s13, const uint8_t* w2, const uint8_t* s2,
              int64_t H, int64_t I, uint16_t* act_row /* [I] */, float* y_row /* [H] */, bool quant = false) {
  std::vector<float> xf(static_cast<size_t>(H));
  for (int64_t h = 0; h < H; ++h) xf[h] = bf16_to_f32(x_row[h]);
  if (quant) quant_row(x_row, H, xf.data(), nullptr, nullptr);
  for (int64_t i = 0; i < I; ++i) {
    ACC g = 0, u = 0;
    for (int64_t h = 0; h < H; ++h) {
      g = g + static_cast<ACC>(weight_value(w13, s13, H, i, h)) * static_cast<ACC>(xf[h]);
      u = u + static_cast<ACC>(weight_value(w13, s13, H, I + i, h)) * static_cast<ACC>(xf[h]);
    }
    const float gf = static_cast<float>(g), uf = static_cast<float>(u);
    const float silu = gf / (1.0f + std::exp(-gf));
    act_row[i] = f32_to_bf16(silu * uf);
  }
  std::vector<float> af(static_cast<size_t>(I));
  for (int64_t i = 0; i < I; ++i) af[i] = bf16_to_f32(act_row[i]);
  if (quant) quant_row(act_row, I, af.data(), nullptr, nullptr);
  for (int64_t n = 0; n < H; ++n) {
    ACC acc = 0;
    for (int64_t i = 0; i < I; ++i)
      acc = acc + static_cast<ACC>(weight_value(w2, s2, I, n, i)) * static_cast<ACC>(af[i]);
    y_row[n] = static_cast<float>(acc);
  }
}

}  // namespace

extern "C" {

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void oracle_set_num_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

float oracle_e2m1_value(int code) { return e2m1_value(static_cast<unsigned>(code) & 0xFu); }
float oracle_e8m0_value(int b) { return e8m0_value(static_cast<unsigned>(b) & 0xFFu); }
float oracle_exp_spec(float d) { return exp_spec(d); }
uint16_t oracle_f32_to_bf16(float f) { return f32_to_bf16(f); }
float oracle_bf16_to_f32(uint16_t h) { return bf16_to_f32(h); }

// Dequantise one matrix [rows, K] to fp32 (used by the tests to hand numpy the
// same logical matrix; the decode itself is pinned against the printed table).
void oracle_dequant(const uint8_t* codes, const uint8_t* scales, int64_t rows, int64_t K, float* out) {
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t h = 0; h < K; ++h) out[r * K + h] = weight_value(codes, scales, K, r, h);
}

// Step a1-a3: ids[T,k], w[T,k], offsets[E+1] (histogram of ids + exclusive scan).
void oracle_route(const float* logits, int T, int E, int k, int32_t* ids, float* w, int32_t* offsets) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t)
    route_token(logits + static_cast<int64_t>(t) * E, E, k, ids + static_cast<int64_t>(t) * k,
                w + static_cast<int64_t>(t) * k);
  std::vector<int64_t> cnt(static_cast<size_t>(E), 0);
  for (int64_t s = 0; s < static_cast<int64_t>(T) * k; ++s) cnt[ids[s]] += 1;
  int64_t run = 0;
  for (int e = 0; e < E; ++e) {
    offsets[e] = static_cast<int32_t>(run);
    run += cnt[e];
  }
  offsets[E] = static_cast<int32_t>(run);
}

// Step a4: stable counting sort of the flat slots s = t*k + j by expert id
// (reading G8): perm[p] = slot at sorted position p, inv_perm[perm[p]] = p,
// x_perm[p,:] = x[perm[p] / k, :].
void oracle_permute(const uint16_t* x, const int32_t* ids, const int32_t* offsets, int T, int H, int E, int k,
                    uint16_t* x_perm, int32_t* perm, int32_t* inv_perm) {
  std::vector<int32_t> next(offsets, offsets + E);
  const int64_t S = static_cast<int64_t>(T) * k;
  for (int64_t s = 0; s < S; ++s) {
    const int32_t p = next[ids[s]]++;
    perm[p] = static_cast<int32_t>(s);
    inv_perm[s] = p;
  }
  if (x_perm != nullptr) {
    for (int64_t p = 0; p < S; ++p)
      std::memcpy(x_perm + p * H, x + static_cast<int64_t>(perm[p] / k) * H, static_cast<size_t>(H) * 2);
  }
}

// Steps a5-a7 over sorted rows.  act may be NULL.  Weight tensors are the
// logical ones: w13[E,2I,H/2], s13[E,2I,H/32], w2[E,H,I/2], s2[E,H,I/32].
static void expert_ffn_rows(const uint16_t* x_perm, const int32_t* offsets, const uint8_t* w13, const uint8_t* s13,
                            const uint8_t* w2, const uint8_t* s2, int T, int H, int I, int E, int k, int acc64, bool quant,
                            uint16_t* act /* [T*k, I] or NULL */, float* y_perm /* [T*k, H] */) {
  const int64_t S = static_cast<int64_t>(T) * k;
  std::vector<int32_t> expert_of(static_cast<size_t>(S));
  for (int e = 0; e < E; ++e)
    for (int32_t p = offsets[e]; p < offsets[e + 1]; ++p) expert_of[p] = e;
  const int64_t w13_e = static_cast<int64_t>(2) * I * (H / 2), s13_e = static_cast<int64_t>(2) * I * (H / 32);
  const int64_t w2_e = static_cast<int64_t>(H) * (I / 2), s2_e = static_cast<int64_t>(H) * (I / 32);
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t p = 0; p < S; ++p) {
    const int e = expert_of[p];
    std::vector<uint16_t> act_row(static_cast<size_t>(I));
    if (acc64)
      ffn_slot<double>(x_perm + p * H, w13 + e * w13_e, s13 + e * s13_e, w2 + e * w2_e, s2 + e * s2_e, H, I,
                       act_row.data(), y_perm + p * H, quant);
    else
      ffn_slot<float>(x_perm + p * H, w13 + e * w13_e, s13 + e * s13_e, w2 + e * w2_e, s2 + e * s2_e, H, I,
                      act_row.data(), y_perm + p * H, quant);
    if (act != nullptr) std::memcpy(act + p * I, act_row.data(), static_cast<size_t>(I) * 2);
  }
}

void oracle_expert_ffn(const uint16_t* x_perm, const int32_t* offsets, const uint8_t* w13, const uint8_t* s13,
                       const uint8_t* w2, const uint8_t* s2, int T, int H, int I, int E, int k, int acc64,
                       uint16_t* act /* [T*k, I] or NULL */, float* y_perm /* [T*k, H] */) {
  expert_ffn_rows(x_perm, offsets, w13, s13, w2, s2, T, H, I, E, k, acc64, false, act, y_perm);
}

// The quantised-activation variant of steps a5-a7 (see quant_block).  `act` receives the intermediate as bf16, i.e.
// before its quantisation.
void oracle_expert_ffn_q(const uint16_t* x_perm, const int32_t* offsets, const uint8_t* w13, const uint8_t* s13,
                         const uint8_t* w2, const uint8_t* s2, int T, int H, int I, int E, int k, int acc64,
                         uint16_t* act /* [T*k, I] or NULL */, float* y_perm /* [T*k, H] */) {
  expert_ffn_rows(x_perm, offsets, w13, s13, w2, s2, T, H, I, E, k, acc64, true, act, y_perm);
}

// Rows of K bf16 values (K a multiple of 32) -> packed codes [rows, K/2], scale bytes [rows, K/32] and the decoded
// values [rows, K]; any output may be NULL.
void oracle_quant_act(const uint16_t* v, int64_t rows, int64_t K, uint8_t* packed, uint8_t* scales, float* deq) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    std::vector<float> d(static_cast<size_t>(K));
    quant_row(v + r * K, K, d.data(), packed != nullptr ? packed + r * (K / 2) : nullptr,
              scales != nullptr ? scales + r * (K / 32) : nullptr);
    if (deq != nullptr) std::memcpy(deq + r * K, d.data(), static_cast<size_t>(K) * 4);
  }
}

// Step a8: out[t,n] = bf16( fma(w_{k-1}, y_{k-1}, ... fma(w_0, y_0, 0)) ), slot
// order j = 0..k-1 (readings G5, G7).  out_f32 may be NULL.
void oracle_combine(const float* y_perm, const int32_t* inv_perm, const float* w, int T, int H, int k,
                    uint16_t* out_bf16, float* out_f32) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    for (int n = 0; n < H; ++n) {
      float acc = 0.0f;
      for (int j = 0; j < k; ++j) {
        const int64_t p = inv_perm[static_cast<int64_t>(t) * k + j];
        acc = std::fmaf(w[static_cast<int64_t>(t) * k + j], y_perm[p * H + n], acc);
      }
      out_bf16[static_cast<int64_t>(t) * H + n] = f32_to_bf16(acc);
      if (out_f32 != nullptr) out_f32[static_cast<int64_t>(t) * H + n] = acc;
    }
  }
}

// ---- the steps either side of the routed path (figure "Execution structure": router scores before the Top-k, the
// shared expert beside the routed experts, "add partials" after them) ----

// Router projection: logits[t,e] = sum over h ascending of x[t,h] * w_router[e,h], both bf16, accumulated in fp32
// (each product of two bf16 values is exact in fp32; only the running sum rounds).  The paper kept a vendor BLAS for
// this step and states no precision; fp32 accumulation of exact products is the reading taken.
void oracle_router_logits(const uint16_t* x, const uint16_t* w_router, int T, int H, int E, float* logits) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    for (int e = 0; e < E; ++e) {
      float acc = 0.0f;
      for (int h = 0; h < H; ++h) {
        const float prod = bf16_to_f32(x[static_cast<int64_t>(t) * H + h]) * bf16_to_f32(w_router[static_cast<int64_t>(e) * H + h]);
        acc = acc + prod;
      }
      logits[static_cast<int64_t>(t) * E + e] = acc;
    }
  }
}

// The join: the routed experts' slot-ordered fp32 sum (exactly oracle_combine's recurrence) plus the shared expert's
// fp32 row, one fp32 addition, then one rounding to bf16.  y_shared[t,:] is the shared expert's down projection of
// token t (the same expert arithmetic as a routed expert, applied to every token with weight 1).
void oracle_combine_shared(const float* y_perm, const int32_t* inv_perm, const float* w, const float* y_shared, int T,
                           int H, int k, uint16_t* out_bf16, float* out_f32) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    for (int n = 0; n < H; ++n) {
      float acc = 0.0f;
      for (int j = 0; j < k; ++j) {
        const int64_t p = inv_perm[static_cast<int64_t>(t) * k + j];
        acc = std::fmaf(w[static_cast<int64_t>(t) * k + j], y_perm[p * H + n], acc);
      }
      acc = acc + y_shared[static_cast<int64_t>(t) * H + n];
      out_bf16[static_cast<int64_t>(t) * H + n] = f32_to_bf16(acc);
      if (out_f32 != nullptr) out_f32[static_cast<int64_t>(t) * H + n] = acc;
    }
  }
}

// The layer by its per-token definition, with no permutation at all: for each
// listed token route it, evaluate its k experts and reduce in slot order.
// Outputs are indexed by position in `tokens`.  y_slots (may be NULL) receives
// the k fp32 per-slot rows of each token, act_slots (may be NULL) the bf16
// activations.  Used for brute-force pins and for sampled parity checks at
// sizes where evaluating every token on the CPU would take hours.
void oracle_forward_tokens(const float* logits, const uint16_t* x, const uint8_t* w13, const uint8_t* s13,
                           const uint8_t* w2, const uint8_t* s2, int T, int H, int I, int E, int k, int acc64,
                           const int32_t* tokens, int n_tokens, int32_t* ids_out /* [n,k] or NULL */,
                           float* w_out /* [n,k] or NULL */, uint16_t* act_slots /* [n,k,I] or NULL */,
                           float* y_slots /* [n,k,H] or NULL */, uint16_t* out_bf16 /* [n,H] */,
                           float* out_f32 /* [n,H] or NULL */) {
  (void)T;
  const int64_t w13_e = static_cast<int64_t>(2) * I * (H / 2), s13_e = static_cast<int64_t>(2) * I * (H / 32);
  const int64_t w2_e = static_cast<int64_t>(H) * (I / 2), s2_e = static_cast<int64_t>(H) * (I / 32);
  std::vector<int32_t> ids(static_cast<size_t>(n_tokens) * k);
  std::vector<float> w(static_cast<size_t>(n_tokens) * k);
  for (int q = 0; q < n_tokens; ++q)
    route_token(logits + static_cast<int64_t>(tokens[q]) * E, E, k, ids.data() + static_cast<int64_t>(q) * k,
                w.data() + static_cast<int64_t>(q) * k);
  std::vector<float> y(static_cast<size_t>(n_tokens) * k * H);
  const int64_t NS = static_cast<int64_t>(n_tokens) * k;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t qs = 0; qs < NS; ++qs) {
    const int64_t q = qs / k;
    const int e = ids[qs];
    std::vector<uint16_t> act_row(static_cast<size_t>(I));
    const uint16_t* x_row = x + static_cast<int64_t>(tokens[q]) * H;
    if (acc64)
      ffn_slot<double>(x_row, w13 + e * w13_e, s13 + e * s13_e, w2 + e * w2_e, s2 + e * s2_e, H, I, act_row.data(),
                       y.data() + qs * H);
    else
      ffn_slot<float>(x_row, w13 + e * w13_e, s13 + e * s13_e, w2 + e * w2_e, s2 + e * s2_e, H, I, act_row.data(),
                      y.data() + qs * H);
    if (act_slots != nullptr) std::memcpy(act_slots + qs * I, act_row.data(), static_cast<size_t>(I) * 2);
  }
  for (int q = 0; q < n_tokens; ++q) {
    for (int n = 0; n < H; ++n) {
      float acc = 0.0f;
      for (int j = 0; j < k; ++j)
        acc = std::fmaf(w[static_cast<int64_t>(q) * k + j], y[(static_cast<int64_t>(q) * k + j) * H + n], acc);
      out_bf16[static_cast<int64_t>(q) * H + n] = f32_to_bf16(acc);
      if (out_f32 != nullptr) out_f32[static_cast<int64_t>(q) * H + n] = acc;
    }
  }
  if (ids_out != nullptr) std::memcpy(ids_out, ids.data(), ids.size() * sizeof(int32_t));
  if (w_out != nullptr) std::memcpy(w_out, w.data(), w.size() * sizeof(float));
  if (y_slots != nullptr) std::memcpy(y_slots, y.data(), y.size() * sizeof(float));
}

}  // extern "C"
