// Shared device helpers of libffint8: status bits, the SUQ scale pair, the counter-based
// rounding hash and the INT8 rounding step (symmetric uniform quantisation, Sec. IV; stochastic
// rounding of Sec. IV-B).  Every FP32 operation on the state path is a single round-to-nearest
// IEEE operation (explicit __f*_rn intrinsics; the library is also built with -fmad=false).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace ffi8 {

// device status word bits (OR-ed by kernels, read by ff_poll_status)
constexpr uint32_t ST_NONFINITE = 1u;
constexpr uint32_t ST_TIMEOUT = 2u;
constexpr uint32_t ST_BADLABEL = 4u;   // a label outside [0, n_classes) met by the label-embedding kernel
constexpr uint32_t ST_RANGE = 8u;      // a weight-gradient sum left the INT32 range (Sec. IV-B: INT32 accumulation)

// Longest contraction whose INT8 x INT8 products cannot leave INT32 whatever the codes: 127*127*n <= 2^31 - 1.
// Longer weight-gradient contractions (convolutions sum over every position of a set) are cut into parts of at
// most this length; the parts are added in 64 bits and a sum outside INT32 raises ST_RANGE.
constexpr long long WG_SAFE_LEN = ((1LL << 31) - 1) / (127LL * 127LL);   // 133144

constexpr int ROUND_NEAREST = 0;
constexpr int ROUND_STOCHASTIC = 1;

constexpr int ROLE_X = 0;
constexpr int ROLE_W = 1;
constexpr int ROLE_DH = 2;

struct RoundKey {
  uint32_t k0, k1;
};

// SplitMix64 output function (key derivation).
__host__ __device__ inline uint64_t splitmix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  uint64_t z = x;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// The values of a train step that change from call to call.  They live in device memory (written by
// set_step_kernel before the step's kernels) instead of kernel arguments, so that the launch sequence
// of a step is the same every time and can be replayed from a captured CUDA graph.
struct StepState {
  unsigned long long step;  // keys the stochastic rounding
  float lambda;             // look-ahead weight of Eq. 3
  float pad;
};

// Key of one quantiser call: the step-independent part (seed, tensor role, layer) is folded on the host,
// the step is folded in on the device.
struct KeySpec {
  unsigned long long s1;
  const StepState* ss;
};
__host__ inline KeySpec make_key_spec(uint64_t seed, int role, int layer, const StepState* ss) {
  uint64_t s0 = splitmix64(seed);
  KeySpec k;
  k.s1 = splitmix64(s0 ^ (uint64_t)((uint32_t)(role & 0xFF) | ((uint32_t)(layer & 0xFFFFFF) << 8)));
  k.ss = ss;
  return k;
}
__device__ __forceinline__ RoundKey derive_key(KeySpec ks) {
  const uint64_t s2 = splitmix64(ks.s1 ^ ks.ss->step);
  RoundKey k;
  k.k0 = (uint32_t)(s2 & 0xFFFFFFFFull);
  k.k1 = (uint32_t)(s2 >> 32);
  return k;
}
// How a dequantised weight gradient g becomes a weight change (Alg. 1, update step names no optimiser):
// kind 0: plain SGD, or heavy ball when Mom is given (m = mu*m + g, W -= lr*m);
// kind 1: Adam - m = b1*m + (1-b1)*g, v = b2*v + (1-b2)*g*g, W -= lr*(m*c1)/(sqrt(v*c2) + eps), with the
// bias corrections c_i = float(1/(1 - b_i^t)), t = step + 1, from FP64 powers taken by square-and-multiply
// from the low bit up (a fixed order of correctly rounded products).  Every FP32 operation is rounded once.
struct UpdateRule {
  int kind;
  float lr, mu, beta2, eps;  // mu: heavy-ball coefficient or Adam's b1
  float* Mom;
  float* Var;
  const StepState* ss;       // Adam reads the step counter here
};
__device__ __forceinline__ double pow_int_rn(double x, unsigned long long n) {
  double r = 1.0, p = x;
  while (n) {
    if (n & 1ull) r = __dmul_rn(r, p);
    n >>= 1;
    if (n) p = __dmul_rn(p, p);
  }
  return r;
}
struct UpdateCoefs {
  float c1, c2, omb1, omb2;
};
__device__ __forceinline__ UpdateCoefs update_coefs(const UpdateRule& r) {
  UpdateCoefs c = {1.0f, 1.0f, 0.0f, 0.0f};
  if (r.kind == 1) {
    const unsigned long long t = r.ss->step + 1ull;
    c.c1 = __double2float_rn(__ddiv_rn(1.0, __dsub_rn(1.0, pow_int_rn((double)r.mu, t))));
    c.c2 = __double2float_rn(__ddiv_rn(1.0, __dsub_rn(1.0, pow_int_rn((double)r.beta2, t))));
    c.omb1 = __fsub_rn(1.0f, r.mu);
    c.omb2 = __fsub_rn(1.0f, r.beta2);
  }
  return c;
}
// New weight for gradient g; m / v are the element's buffer values, rewritten when the rule uses them.
__device__ __forceinline__ float apply_update(const UpdateRule& r, const UpdateCoefs& c, float w, float g, float& m, float& v) {
  if (r.kind == 1) {
    m = __fadd_rn(__fmul_rn(r.mu, m), __fmul_rn(c.omb1, g));
    v = __fadd_rn(__fmul_rn(r.beta2, v), __fmul_rn(c.omb2, __fmul_rn(g, g)));
    const float upd = __fdiv_rn(__fmul_rn(m, c.c1), __fadd_rn(__fsqrt_rn(__fmul_rn(v, c.c2)), r.eps));
    return __fsub_rn(w, __fmul_rn(r.lr, upd));
  }
  if (r.Mom) g = m = __fadd_rn(__fmul_rn(r.mu, m), g);
  return __fsub_rn(w, __fmul_rn(r.lr, g));
}

// Range vectors (8 floats per layer) that the same launch clears for the step that follows.
struct RangeTable {
  float* p[32];
  int n;
};
__global__ void set_step_kernel(StepState* ss, unsigned long long step, float lambda, int set_lambda, RangeTable ranges) {
  if (threadIdx.x == 0) {
    ss->step = step;
    if (set_lambda) ss->lambda = lambda;
  }
  if ((int)threadIdx.x < ranges.n * 8) ranges.p[threadIdx.x >> 3][threadIdx.x & 7] = 0.0f;
}

// s = a/127, inv = 127/a.  A zero tensor, or one whose range is below 2^-100 (127/a would leave
// the FP32 range for subnormal a), quantises to zeros: s = 1, inv = 0.
constexpr float TINY_RANGE = 7.888609052210118e-31f;  // 2^-100
__device__ __forceinline__ float scale_of(float a) {
  return a < TINY_RANGE ? 1.0f : __fdiv_rn(a, 127.0f);
}
__device__ __forceinline__ float inv_of(float a) {
  return a < TINY_RANGE ? 0.0f : __fdiv_rn(127.0f, a);
}

// One 32-bit hash per element PAIR (pair index = linear index >> 1).
__device__ __forceinline__ uint32_t pair_hash(uint32_t pair, RoundKey key) {
  uint32_t h = pair ^ key.k0;
  h *= 0x9E3779B1u;
  h ^= h >> 15;
  h = (h + key.k1) * 0x85EBCA6Bu;
  h ^= h >> 13;
  h *= 0xC2B2AE35u;
  h ^= h >> 16;
  return h;
}
// u in [0,1) with 16 random bits: low half of the pair hash for even indices, high half for odd.
// u = half16 * 2^-16, formed without shifts or an integer-to-float conversion: floats in [128, 256)
// have an ulp of 2^-16, so the bit pattern 0x4300hhhh is 128 + half16*2^-16 and subtracting 128 is
// exact.  One byte permute places the half (HI = 0: bytes 0-1 of h, HI = 1: bytes 2-3).
template <int HI>
__device__ __forceinline__ float u_from_hash(uint32_t h) {
  const uint32_t bits = __byte_perm(h, 0x43000000u, HI ? 0x7632 : 0x7610);
  return __fsub_rn(__uint_as_float(bits), 128.0f);
}

// rint(t) (ties to even) or floor(t+u), then clip to [-127, 127], as one saturating float-to-int8
// conversion.  |x| <= a gives |t| <= 127 up to one rounding, so: nearest never reaches -128; for
// floor, clamping t at -127 first gives the same result as clipping afterwards (u >= 0), and the
// conversion's saturation at +127 is the upper clip.  MODE is a compile-time constant.
template <int MODE>
__device__ __forceinline__ int round_clip(float t, float u) {
  int r;
  if (MODE == ROUND_NEAREST) {
    asm("cvt.rni.sat.s8.f32 %0, %1;" : "=r"(r) : "f"(t));
  } else {
    const float v = __fadd_rn(fmaxf(t, -127.0f), u);
    asm("cvt.rmi.sat.s8.f32 %0, %1;" : "=r"(r) : "f"(v));
  }
  return r;
}

// Quantise two neighbouring elements (even linear index idx_even and idx_even+1).
template <int MODE>
__device__ __forceinline__ void quant_pair(float x0, float x1, float inv, uint32_t idx_even, RoundKey key, int& q0, int& q1) {
  float u0 = 0.0f, u1 = 0.0f;
  if (MODE != ROUND_NEAREST) {
    const uint32_t h = pair_hash(idx_even >> 1, key);
    u0 = u_from_hash<0>(h);
    u1 = u_from_hash<1>(h);
  }
  q0 = round_clip<MODE>(__fmul_rn(x0, inv), u0);
  q1 = round_clip<MODE>(__fmul_rn(x1, inv), u1);
}
// Quantise one element at an arbitrary linear index.
template <int MODE>
__device__ __forceinline__ int quant_one(float x, float inv, uint32_t idx, RoundKey key) {
  float u = 0.0f;
  if (MODE != ROUND_NEAREST) {
    const uint32_t h = pair_hash(idx >> 1, key);
    u = (idx & 1u) ? u_from_hash<1>(h) : u_from_hash<0>(h);
  }
  return round_clip<MODE>(__fmul_rn(x, inv), u);
}

// Low bytes of four ints as one little-endian word (three byte permutes).
__device__ __forceinline__ uint32_t pack4(int q0, int q1, int q2, int q3) {
  const uint32_t lo = __byte_perm((uint32_t)q0, (uint32_t)q1, 0x0040);
  const uint32_t hi = __byte_perm((uint32_t)q2, (uint32_t)q3, 0x0040);
  return __byte_perm(lo, hi, 0x5410);
}

__device__ __forceinline__ float dequant_relu(int acc, float c) {
  return fmaxf(0.0f, __fmul_rn(__int2float_rn(acc), c));
}

}  // namespace ffi8
