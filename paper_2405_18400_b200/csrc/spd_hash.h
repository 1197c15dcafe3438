// Slot format and hash of the n-gram tables; the one piece the host-side builder and the device-side
// probe must agree on.  A slot is 16 bytes: six uint16 token ids packed into three 32-bit words
// (token 2i in the low half of word i), then a uint32 count; count 0 marks an empty slot.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define SPD_HD __host__ __device__ __forceinline__
#else
#define SPD_HD inline
#endif

struct SpdSlot {
  uint32_t w0, w1, w2, count;
};

SPD_HD uint64_t spd_key_hash(uint32_t w0, uint32_t w1, uint32_t w2) {
  uint64_t x = (((uint64_t)w1 << 32) | (uint64_t)w0) ^ ((uint64_t)w2 * 0x9E3779B97F4A7C15ull);
  x ^= x >> 32;
  x *= 0xD6E8FEB86659FD93ull;
  x ^= x >> 32;
  x *= 0xD6E8FEB86659FD93ull;
  x ^= x >> 32;
  return x;
}

// Packs up to six token ids (tok[0..n)) into the three key words.
SPD_HD void spd_pack_key(const int32_t *tok, int n, uint32_t &w0, uint32_t &w1, uint32_t &w2) {
  uint32_t t[6];
  for (int i = 0; i < 6; ++i) t[i] = i < n ? (uint32_t)tok[i] & 0xffffu : 0u;
  w0 = t[0] | (t[1] << 16);
  w1 = t[2] | (t[3] << 16);
  w2 = t[4] | (t[5] << 16);
}
