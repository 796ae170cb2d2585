// The random vectors f of the locator (Section 3.4: f ~ N(1, I)): f_n[kappa][p] = 1 + N(0, 1), draw n of a plan's seed.
// Philox4x32-7 (seven rounds: the smallest count its authors found to pass every statistical test battery; the
// vectors need an absolutely continuous law, not cryptographic strength) with counter (quad index low, high, kappa | high word of n << 8, low word of n) and key = seed gives four
// 32-bit words per quad of consecutive coordinates; Box-Muller turns them into four normal values.
#pragma once

#include <stdint.h>

namespace solon {

__device__ __forceinline__ void philox4x32_7(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t out[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int round = 0; round < 7; ++round) {
    uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    uint32_t n0 = hi1 ^ c1 ^ k0, n1 = lo1, n2 = hi0 ^ c3 ^ k1, n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0;
    k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Coordinates 4 quad .. 4 quad + 3 of f_n[kappa]; entries at or beyond d_c (the padding of the row pitch) are zero.
// Box-Muller with the fast logarithm and sine/cosine: any absolutely continuous law will do for f, and the vectors are
// only ever read back from memory, never regenerated elsewhere.
__device__ __forceinline__ float4 projection_quad(uint64_t seed, unsigned long long n, int kappa, int64_t quad, int64_t d_c) {
  uint32_t x[4];
  philox4x32_7((uint32_t)quad, (uint32_t)(quad >> 32), (uint32_t)kappa | ((uint32_t)(n >> 32) << 8), (uint32_t)n, (uint32_t)seed,
                (uint32_t)(seed >> 32), x);
  float v[4];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    float u1 = ((float)x[2 * h] + 0.5f) * 2.3283064365386963e-10f;       // (0, 1]
    const float u2 = ((float)x[2 * h + 1] + 0.5f) * 2.3283064365386963e-10f;
    u1 = fminf(fmaxf(u1, 1.0e-12f), 1.0f);
    const float rad = sqrtf(-2.0f * __logf(u1));
    float sn, cs;
    __sincosf(6.283185307179586f * u2, &sn, &cs);
    v[2 * h] = 1.0f + rad * cs;
    v[2 * h + 1] = 1.0f + rad * sn;
  }
  float4 out;
  out.x = (quad * 4 + 0 < d_c) ? v[0] : 0.0f;
  out.y = (quad * 4 + 1 < d_c) ? v[1] : 0.0f;
  out.z = (quad * 4 + 2 < d_c) ? v[2] : 0.0f;
  out.w = (quad * 4 + 3 < d_c) ? v[3] : 0.0f;
  return out;
}

// What the vectors' generator needs: both buffers (draw n lives in buffer n & 1), shape, seed, and the device-side count.
struct DrawParams {
  float* f[2];
  int64_t d_c, pitch;
  int K;
  uint64_t seed;
  unsigned long long* draw;     // [0] index of the draw the next projection kernel reads, [1] ticket
};

// Write draw (draw[0] + advance) into its buffer with the calling CTAs cta = 0 .. n_ctas - 1 of n_threads threads each; with
// advance = 1 the last CTA to finish (atomic ticket; every CTA has read draw[0] by then) makes it the current draw.
__device__ __forceinline__ void draw_projection_vectors(const DrawParams& dp, int advance, int cta, int n_ctas, int tid, int n_threads) {
  const unsigned long long n = dp.draw[0] + (unsigned long long)advance;
  float* f = dp.f[n & 1ULL];
  const int64_t quads = (dp.d_c + 3) / 4;
  const int64_t total = quads * dp.K;
  for (int64_t i = (int64_t)cta * n_threads + tid; i < total; i += (int64_t)n_ctas * n_threads) {
    const int kappa = (int)(i / quads);
    const int64_t quad = i - (int64_t)kappa * quads;
    *reinterpret_cast<float4*>(f + (int64_t)kappa * dp.pitch + quad * 4) = projection_quad(dp.seed, n, kappa, quad, dp.d_c);
  }
  if (advance) {
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      if (atomicAdd(dp.draw + 1, 1ULL) == (unsigned long long)n_ctas - 1) {
        dp.draw[1] = 0ULL;
        dp.draw[0] = n;
      }
    }
  }
}

}  // namespace solon
