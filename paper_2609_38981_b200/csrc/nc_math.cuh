// The numerical contract: every scalar operation whose rounding decides output
// bits, written once with explicit round-to-nearest intrinsics so that no two
// kernels can contract or reassociate it differently.
//
// Per (request, position p, query head) the output bits are a function of the
// query row, the logical keys/values 0..p, the scale and these constants only:
//   * key tiles are absolute: tile t covers keys [64 t, 64 t + 64) counted from
//     position 0 of the request (App. A, tile IR: t = 0..N-1, j = t*B_N + b);
//   * KV splits are absolute too: split k covers [512 k, 512 k + 512); inside a
//     split the state (m, z, U) starts at (-inf, 0, 0) and is updated tile by
//     tile in ascending order exactly as in the paper's iteration;
//   * split results are folded left to right by split index.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace vosti {
namespace nc {

constexpr int kKeyTile = 64;        // B_N
constexpr int kSplitLen = 512;      // L_S, a multiple of B_N
constexpr int kTilesPerSplit = kSplitLen / kKeyTile;
constexpr int kRowsPerGroup = 16;   // rows packed into one MMA row tile
constexpr int kSplitRowsMax = 32;   // requests with at most this many rows per KV head run split-parallel
constexpr int kPageSize = 16;
constexpr int kPagesPerTile = kKeyTile / kPageSize;
constexpr int kPagesPerSplit = kSplitLen / kPageSize;
constexpr uint32_t kVersion = 2;

// Rule ids: every choice below that decides output bits has a name and a value here, and
// vosti_fingerprint hashes all of them (a changed rule must change its value).
constexpr uint32_t kRuleExponent = 1;   // A = ex2.approx.ftz(fma(S, c, -m_hat)), alpha = ex2.approx.ftz(m - m_hat)
constexpr uint32_t kRuleMaximum = 2;    // lazy reference maximum: m_hat moves only when the tile's scaled maximum
                                        // exceeds m by more than kLazyMaxStep (1 would be the exact running maximum)
constexpr uint32_t kRuleRowSum = 3;     // per half of 32 lanes: eight chains over b mod 8, pairs, (P0 + P1) + (P2 + P3); lower + upper
constexpr uint32_t kRuleFold = 1;       // left fold by split index: z = fma(z_c, a, z_k * b), U likewise
constexpr uint32_t kRuleReciprocal = 1; // 1 / z by rcp.rn, O = U * inv
constexpr uint32_t kRuleZeroSign = 1;   // O + 0.0: an exact zero is +0
constexpr uint32_t kRuleMmaChunks = 1;  // bf16 x bf16 -> fp32, chunks of 16 ascending, fresh accumulator per tile / split
constexpr uint32_t kRuleLse = 1;        // (m + lg2.approx.ftz(z)) * ln 2
constexpr float kLazyMaxStep = 8.0f;    // base-two domain: weights stay below 2^8

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Reference maximum in the scaled (base-two) domain.  The raw maximum is taken
// over visible lanes first; multiplying by c >= 0 is monotone, so its product
// with c is the maximum of the scaled scores.  The reference is LAZY: it moves
// to the tile's maximum only when that exceeds it by more than kLazyMaxStep, so
// that in the common case alpha is exactly 1 and U needs no rescale.  Any
// reference within a bounded distance of the true maximum gives the same
// quotient U / z up to rounding; this one keeps every weight below 2^8.  The
// first visible tile of a split always sets it (m_old = -inf).
__device__ __forceinline__ float new_max(float m_old, float raw_max_visible, float c) {
  const float t = __fmul_rn(raw_max_visible, c);
  return t > __fadd_rn(m_old, kLazyMaxStep) ? t : m_old;
}
// alpha = 2^(m - m_hat); ex2(0) is exactly 1, so the unchanged case needs no instruction
__device__ __forceinline__ float rescale(float m_old, float m_new) {
  return m_old == m_new ? 1.0f : ex2(__fsub_rn(m_old, m_new));
}
// A = 2^(s*c - m_hat), one fused multiply-add then the exponential.
__device__ __forceinline__ float weight(float s, float c, float neg_m_new) {
  return ex2(__fmaf_rn(s, c, neg_m_new));
}
// z_hat = z*alpha + sum_b A
__device__ __forceinline__ float z_update(float z, float alpha, float row_sum) {
  return __fmaf_rn(z, alpha, row_sum);
}
__device__ __forceinline__ float u_rescale(float u, float alpha) { return __fmul_rn(u, alpha); }

// sum_b A over the 64 lanes of a tile, order fixed by the lane index b alone.  The tile is
// taken as two halves of 32 lanes (b < 32, b >= 32).  Within a half: eight chains, chain j
// takes the lanes with b mod 8 == j in ascending b (four lanes each); pair q = chain 2q +
// chain 2q+1; half sum = (pair0 + pair1) + (pair2 + pair3).  Tile sum = lower half + upper half.
// `a` holds the sixteen lanes of one pair over the whole tile: a[2n] = lane 8n + 2q,
// a[2n+1] = lane 8n + 2q + 1; HALF selects n = 0..3 or n = 4..7.
template <int HALF>
__device__ __forceinline__ float quad_partial(const float (&a)[16]) {
  float e0 = a[8 * HALF], e1 = a[8 * HALF + 1];
#pragma unroll
  for (int n = 1; n < 4; ++n) {
    e0 = __fadd_rn(e0, a[8 * HALF + 2 * n]);
    e1 = __fadd_rn(e1, a[8 * HALF + 2 * n + 1]);
  }
  return __fadd_rn(e0, e1);
}
__device__ __forceinline__ float quad_total(float s0, float s1, float s2, float s3) {
  return __fadd_rn(__fadd_rn(s0, s1), __fadd_rn(s2, s3));
}
__device__ __forceinline__ float tile_total(float lower_half, float upper_half) { return __fadd_rn(lower_half, upper_half); }

// Two lanes at a time.  Each half of a packed f32x2 operation is the same IEEE
// round-to-nearest operation as its scalar form above, so a kernel may use
// either form for any lane without changing a bit; the packed forms halve the
// instruction count where one thread owns many lanes of a row.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// A for two lanes: 2^(s*c - m_hat) each.
__device__ __forceinline__ void weight2(float s0, float s1, uint64_t c2, uint64_t neg_m2, float& a0, float& a1) {
  float e0, e1;
  unpack2(fma2(pack2(s0, s1), c2, neg_m2), e0, e1);
  a0 = ex2(e0);
  a1 = ex2(e1);
}
// maximum of three (the maximum is order-free; inputs are finite or -inf)
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Left fold of split results.  (m_c, z_c, U_c) <- fold((m_c, z_c, U_c), (m_k, z_k, U_k)).
struct FoldFactors {
  float a, b;
};
__device__ __forceinline__ FoldFactors fold_scalars(float& m_c, float& z_c, float m_k, float z_k) {
  const float m_star = fmaxf(m_c, m_k);
  FoldFactors f;
  f.a = ex2(__fsub_rn(m_c, m_star));
  f.b = ex2(__fsub_rn(m_k, m_star));
  z_c = __fmaf_rn(z_c, f.a, __fmul_rn(z_k, f.b));
  m_c = m_star;
  return f;
}
__device__ __forceinline__ float fold_u(float u_c, float u_k, FoldFactors f) {
  return __fmaf_rn(u_c, f.a, __fmul_rn(u_k, f.b));
}

// O = U * select(z > 0, 1/z, 0); adding +0 turns a -0 result into +0 so that
// the sign of an exactly-zero output cannot depend on which masked lanes a
// schedule happened to multiply by zero.
__device__ __forceinline__ float out_scale(float z) { return z > 0.0f ? __frcp_rn(z) : 0.0f; }
__device__ __forceinline__ float out_value(float u, float inv) {
  return __fadd_rn(__fmul_rn(u, inv), 0.0f);
}

// Auxiliary log-sum-exp of the scaled scores, natural logarithm: (m + log2 z) ln 2.
__device__ __forceinline__ float lse_value(float m, float z) {
  float l;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(l) : "f"(z));
  return __fmul_rn(__fadd_rn(m, l), 0.693147180559945309f);
}

// Sliding window (App. A: "adds j > p - w"): the row at p sees keys lo < j <= p with
// lo = p - w; without a window lo lies below every key.  Padding rows (p = -1) see nothing.
constexpr int kNoLowerBound = -0x40000000;
__device__ __forceinline__ int window_lo(int p, int window) {
  return (window > 0 && p >= 0) ? p - window : kNoLowerBound;
}
// First key tile / split a row (or a group whose first row is at p) needs.
__device__ __forceinline__ int first_key(int p, int window) {
  return (window > 0 && p - window + 1 > 0) ? p - window + 1 : 0;
}

}  // namespace nc
}  // namespace vosti
