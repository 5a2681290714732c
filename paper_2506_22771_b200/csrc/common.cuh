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

constexpr int ROUND_NEAREST = 0;
constexpr int ROUND_STOCHASTIC = 1;

constexpr int ROLE_X = 0;
constexpr int ROLE_W = 1;
constexpr int ROLE_DH = 2;

struct RoundKey {
  uint32_t k0, k1;
};

// SplitMix64 output function (host side key derivation).
__host__ inline uint64_t splitmix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  uint64_t z = x;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__host__ inline RoundKey make_round_key(uint64_t seed, int role, int layer, uint64_t step) {
  uint64_t s0 = splitmix64(seed);
  uint64_t s1 = splitmix64(s0 ^ (uint64_t)((uint32_t)(role & 0xFF) | ((uint32_t)(layer & 0xFFFFFF) << 8)));
  uint64_t s2 = splitmix64(s1 ^ step);
  RoundKey k;
  k.k0 = (uint32_t)(s2 & 0xFFFFFFFFull);
  k.k1 = (uint32_t)(s2 >> 32);
  return k;
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
__device__ __forceinline__ float u_from_half(uint32_t half16) {
  return __fmul_rn(__uint2float_rn(half16), 1.52587890625e-05f);  // * 2^-16, exact
}

__device__ __forceinline__ int round_clip(float t, float u, int mode) {
  float r = (mode == ROUND_NEAREST) ? rintf(t) : floorf(__fadd_rn(t, u));
  r = fminf(fmaxf(r, -127.0f), 127.0f);
  return __float2int_rn(r);
}

// Quantise two neighbouring elements (even linear index idx_even and idx_even+1).
__device__ __forceinline__ void quant_pair(float x0, float x1, float inv, int mode, uint32_t idx_even,
                                           RoundKey key, int& q0, int& q1) {
  float u0 = 0.0f, u1 = 0.0f;
  if (mode != ROUND_NEAREST) {
    uint32_t h = pair_hash(idx_even >> 1, key);
    u0 = u_from_half(h & 0xFFFFu);
    u1 = u_from_half(h >> 16);
  }
  q0 = round_clip(__fmul_rn(x0, inv), u0, mode);
  q1 = round_clip(__fmul_rn(x1, inv), u1, mode);
}
// Quantise one element at an arbitrary linear index.
__device__ __forceinline__ int quant_one(float x, float inv, int mode, uint32_t idx, RoundKey key) {
  float u = 0.0f;
  if (mode != ROUND_NEAREST) {
    uint32_t h = pair_hash(idx >> 1, key);
    u = u_from_half((idx & 1u) ? (h >> 16) : (h & 0xFFFFu));
  }
  return round_clip(__fmul_rn(x, inv), u, mode);
}

__device__ __forceinline__ uint32_t pack4(int q0, int q1, int q2, int q3) {
  return (uint32_t)(q0 & 0xFF) | ((uint32_t)(q1 & 0xFF) << 8) | ((uint32_t)(q2 & 0xFF) << 16) |
         ((uint32_t)(q3 & 0xFF) << 24);
}

__device__ __forceinline__ float dequant_relu(int acc, float c) {
  return fmaxf(0.0f, __fmul_rn(__int2float_rn(acc), c));
}

}  // namespace ffi8
