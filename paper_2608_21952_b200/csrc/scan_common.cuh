// What the two ChunkScan kernels (chunk_scan.cu: int8 masked operand; chunk_scan_f16.cu: the paper's FP16
// operand) share: the walk of a persistent CTA over its (batch, chunk, head) units, the ring indices of the
// CBq and xq buffers, and the exact int8 -> binary32 unpack.
#pragma once
#include "kernels.h"

namespace ssdi8 {
namespace scan {

constexpr uint32_t PANEL = 16384;    // [128][128] int8

// CBq ring of 4: buffers 0,1 hold two panels (32 KB), buffers 2,3 one (16 KB)
__device__ __forceinline__ uint32_t cb_offset(uint32_t off_cb, int idx) {
  return off_cb + (idx < 2 ? (uint32_t)idx * 32768u : 65536u + (uint32_t)(idx - 2) * 16384u);
}
// which CBq buffer tile n of this CTA uses: with two tiles per chunk the second (two panels)
// alternates between buffers 0,1 and the first (one panel) between 2,3; otherwise all four rotate
__device__ __forceinline__ int cb_index(int n, int it, int ntpu) {
  return ntpu == 1 ? (n & 3) : ((it ? 0 : 2) + ((n >> 1) & 1));
}
// the xq buffer of tile n and the phase of its barriers: one buffer per chunk, shared by its tiles
__device__ __forceinline__ int x_index(int n, int ntpu) { return ntpu == 1 ? (n & 1) : ((n >> 1) & 1); }
__device__ __forceinline__ uint32_t x_phase(int n, int ntpu) { return ntpu == 1 ? ((n >> 1) & 1) : ((n >> 2) & 1); }

// two int8 of w_xor (= word ^ 0x80808080), bytes k and k+1, as exact floats
__device__ __forceinline__ float2 unpack2(uint32_t w_xor, int k) {
  const float2 m = make_float2(__uint_as_float(__byte_perm(w_xor, 0x4B400000u, 0x7650u + k)),
                               __uint_as_float(__byte_perm(w_xor, 0x4B400000u, 0x7651u + k)));
  return __fadd2_rn(m, make_float2(-kMagicIn, -kMagicIn));
}

// A CTA walks the units u = blockIdx.x + i gridDim.x (head fastest, then chunk, then batch), both tiles of
// a unit in turn.  The CTAs of the grid therefore work on neighbouring heads of the same tokens at the same
// time: the rows of x they read and the rows of y they write (256 bytes per token and head, the heads of a
// token adjacent in memory) fill whole DRAM pages while they are in L2, and the Cq / CBq tiles of a group
// are fetched once for all its heads.  (With consecutive units per CTA instead, a token's heads were
// written far apart in time and the writes reached DRAM in 256-byte pieces: measured on a copy
// of the int8 kernel with its arithmetic compiled out, 0.125 against 0.115 ms.)
struct UnitWalk {
  int units;        // (batch, chunk, head) units of the launch
  int dh, dk, db;   // the grid size as a step (db, dk, dh) in (batch, chunk, head) mixed radix
  int hpg;          // heads per group
};
struct Tile {
  int b, k, h, it, KJ;
  i64 tok0, unit;              // tok0 = b L + k Q, unit = (b*H + h)*c + k
};
// The step to the CTA's next unit, without divisions (every role walks the tiles, so this is inlined many
// times and runs once per tile on each role's critical path).
__device__ __forceinline__ void next_unit(Tile& x, const Dims& d, const UnitWalk& w) {
  x.h += w.dh;
  x.k += w.dk;
  x.b += w.db;
  if (x.h >= d.H) { x.h -= d.H; ++x.k; }
  if (x.k >= d.c) { x.k -= d.c; ++x.b; }
  x.tok0 = ((i64)x.b * d.c + x.k) * d.Q;      // L = c Q
  x.unit = ((i64)x.b * d.H + x.h) * d.c + x.k;
}
__device__ __forceinline__ void next_tile(Tile& x, const Dims& d, const UnitWalk& w, int TM, int ntpu) {
  if (++x.it == ntpu) {
    x.it = 0;
    next_unit(x, d, w);
  }
  x.KJ = (x.it + 1) * TM;
}
// the first tile of the CTA's next unit
__device__ __forceinline__ void next_head(Tile& x, const Dims& d, const UnitWalk& w, int TM, int ntpu) {
  x.it = ntpu - 1;
  next_tile(x, d, w, TM, ntpu);
}
// first tile of a CTA (unit u)
__device__ __forceinline__ Tile decode_unit(int u, const Dims& d, int TM) {
  Tile x;
  x.it = 0;
  x.h = u % d.H; u /= d.H;
  x.k = u % d.c;
  x.b = u / d.c;
  x.KJ = TM;
  x.tok0 = (i64)x.b * d.L + (i64)x.k * d.Q;
  x.unit = ((i64)x.b * d.H + x.h) * d.c + x.k;
  return x;
}
// tiles of CTA `cta` of a grid of `grid` CTAs: its units cta, cta + grid, ..., ntpu tiles each
__device__ __forceinline__ int tiles_of_cta(const UnitWalk& w, int cta, int grid, int ntpu) {
  return (((w.units - 1 - cta) / grid) + 1) * ntpu;
}

// Host: one CTA per SM; when there are more units than SMs, the grid size is taken coprime with the number of
// heads (a few CTAs fewer at most), so that the heads a CTA meets, h0 + i * grid mod H, run through all
// heads instead of a fraction of them: the mask's work differs from head to head with the decay rate, and
// the kernel ends with its slowest CTA.  Returns false if the launch has too many tiles for 32-bit counters.
inline bool make_unit_walk(const Dims& d, int TM, int sms, UnitWalk* w, int* grid) {
  const i64 units64 = (i64)d.b * d.c * d.H;
  if (units64 * (d.Q / TM) >= ((i64)1 << 30)) return false;
  const int units = (int)units64;
  int g = units < sms ? units : sms;
  if (units > sms) {
    auto gcd = [](int x, int y) { while (y) { const int t = x % y; x = y; y = t; } return x; };
    for (int gtry = g; gtry > g - 8 && gtry > 1; --gtry)
      if (gcd(gtry, d.H) == 1) { g = gtry; break; }
  }
  // the grid size as a step in (batch, chunk, head) mixed radix, head fastest
  *w = UnitWalk{units, g % d.H, (g / d.H) % d.c, g / d.H / d.c, d.H / d.G};
  *grid = g;
  return true;
}

}  // namespace scan
}  // namespace ssdi8
