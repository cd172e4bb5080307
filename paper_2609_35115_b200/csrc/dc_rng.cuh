// Device random streams: Philox4x32-10 (Salmon et al. 2011, "Parallel random numbers: as easy as 1, 2, 3") and the
// map from one draw to four standard normals.  Counter-based: a draw is a pure function of (key, counter), so the
// generator's "offset" is whatever clock the caller puts into the counter - a replayed graph draws what direct
// launches draw (the device-randomness clause of the paper's effect classification, Section 3.3).
#pragma once
#include <stdint.h>

namespace dc {

// Ten rounds of two 32 x 32 -> 64 multiplications and a key bump.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1, uint32_t* out) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Four standard normals from the four words of one draw: two Box-Muller pairs on u = ((r >> 8) + 1/2) 2^-24,
// (w0, w1) -> z0 = r cos, z1 = r sin; (w2, w3) -> z2, z3.
__device__ __forceinline__ void normals4(const uint32_t* w, float* z) {
  const float u0 = ((float)(w[0] >> 8) + 0.5f) * (1.0f / 16777216.0f), u1 = ((float)(w[1] >> 8) + 0.5f) * (1.0f / 16777216.0f);
  const float u2 = ((float)(w[2] >> 8) + 0.5f) * (1.0f / 16777216.0f), u3 = ((float)(w[3] >> 8) + 0.5f) * (1.0f / 16777216.0f);
  const float ra = sqrtf(-2.0f * logf(u0)), rb = sqrtf(-2.0f * logf(u2));
  float sa, ca, sb, cb;
  sincosf(6.283185307179586f * u1, &sa, &ca);
  sincosf(6.283185307179586f * u3, &sb, &cb);
  z[0] = ra * ca; z[1] = ra * sa; z[2] = rb * cb; z[3] = rb * sb;
}

}  // namespace dc
