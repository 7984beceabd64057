// Shared device/host helpers of liblightkv (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lightkv.h"

namespace lkv {

constexpr int kMaxTiles = 32;          // image tiles / frames per sample
constexpr int kFdTile = 128;           // A (and B) entries per tile of the tensor-core FD kernel
constexpr int kMaxWindows = 2048;      // windows per sample (window-build kernel keeps 32 x n_windows u16 counters in smem)
constexpr int kMaxWindowTokens = 65535;  // tokens of one window (range of those counters)

// Grid geometry of one stage, passed by value to the kernels.
struct Geometry {
  int n_tiles;
  int w;                               // windows per axis, per tile
  int n_windows;                       // n_tiles * w * w
  int src_par;                         // parity of the local rank of the source nodes (0: A -> B, 1: B -> A)
  int tile_off[kMaxTiles + 1];         // first flat position of each tile
  int rows[kMaxTiles];
  int cols[kMaxTiles];
};

// Tiling of one sample's A x B pairs for the tensor-core FD kernel.  Consecutive groups of `wpt`
// windows share one tile while every window has at most 128 A entries; larger windows are cut into
// blocks_a x blocks_b blocks of 128 x 128 entries (wpt = 1).  `passes` * 32 bounds the A (and B)
// entries of any tile; the kernel sizes its shared-memory stages from it.
struct FdTiling {
  int n_tiles;                         // groups * blocks_a * blocks_b
  int wpt;                             // windows per group
  int blocks_a, blocks_b;
  int passes;                          // 1, 2 or 4
  int pad[3];
};

// Groups are kept small enough that the whole batch yields about this many tiles (two per SM).
constexpr int kFdTargetTiles = 296;

// Per-stage views into the caller's workspace (all DEVICE pointers, per-sample row strides in elements).
struct Workspace {
  int* win_off;    // [B, n_windows + 1]  first window-sorted slot of each window
  int* a_off;      // [B, n_windows + 1]  first A entry of each window (B entry offset = win_off - a_off)
  int* tok_win;    // [B, cap_in]         window of each token
  int* tok_l;      // [B, cap_in]         local index inside its window (even = A, odd = B)
  int* a_tok;      // [B, cap_a]          token index of each A entry (entries grouped by window)
  int* a_win;      // [B, cap_a]          window of each A entry
  int* b_tok;      // [B, cap_b]          token index of each B entry
  unsigned long long* a_key;  // [B, cap_a]  (orderable(lowest FD) << 32) | B entry index of the best partner;
                              //             all ones while no partner is known (set by the window build)
  FdTiling* fd_tiling;        // [B]         how the tensor-core FD kernel cuts this sample into tiles
  float* xi_h;     // [B, H, cap_in]      per-head attention mass on the prompt (ATTN modes)
  float* xi;       // [B, cap_in]
  int* partner;    // [B, cap_in]         token an A token is merged into, -1 = survives
  int* slot;       // [B, cap_in]         output slot of surviving tokens
  int* a_partner;  // [B, cap_a]          per A entry: token it is merged into, -1 = survives
  unsigned int* xi_sched;   // [4]        ticket counters and list length of the tensor-core xi kernel
  int* xi_redo;    // [ceil(cap_in / 128) * H * B]  its work items that need the second, safe launch
  int cap_in, cap_out, cap_a, cap_b, n_windows;
};

// Prompt-token set J: up to LIGHTKV_MAX_TEXT_RANGES ascending, disjoint ranges of sequence indices in front of
// the vision block.  begin / end bound the whole set.
struct TextSet {
  int n;
  int begin, end;
  int lo[LIGHTKV_MAX_TEXT_RANGES], hi[LIGHTKV_MAX_TEXT_RANGES];
  __host__ __device__ inline bool holds(int j) const {
    for (int i = 0; i < n; ++i)
      if (j >= lo[i] && j < hi[i]) return true;
    return false;
  }
  // bit c set <=> key j0 + c belongs to J (c < 64)
  __host__ __device__ inline unsigned long long mask64(int j0) const {
    unsigned long long m = 0;
    for (int i = 0; i < n; ++i) {
      const int a = (lo[i] > j0 ? lo[i] : j0) - j0, b = (hi[i] < j0 + 64 ? hi[i] : j0 + 64) - j0;
      if (b > a) m |= (b - a >= 64 ? ~0ull : ((1ull << (b - a)) - 1ull)) << a;
    }
    return m;
  }
};

// Tokens removed from a window of n tokens when a fraction `keep` must remain:
// floor((1 - keep) n) evaluated as n - ceil(keep n - 1e-9), at most the number of source nodes (the tokens
// of local rank parity `src_par`: ceil(n / 2) A nodes, or floor(n / 2) B nodes in the reverse direction), none
// from a window of one token.
__host__ __device__ inline int removal_count(int n, double keep, int src_par = 0) {
  if (n < 2) return 0;
#ifdef __CUDA_ARCH__
  double t = __dadd_rn(__dmul_rn(keep, (double)n), -1e-9);
#else
  volatile double prod = keep * (double)n;   // no fused multiply-add on the host either
  double t = prod - 1e-9;
#endif
  int r = n - (int)ceil(t);
  int na = (n + 1 - src_par) >> 1;
  return r < 0 ? 0 : (r > na ? na : r);
}

// Window id of a flat grid position; -1 when the position lies outside every tile.
__host__ __device__ inline int window_of(const Geometry& g, int pos) {
  int t = -1;
  for (int i = 0; i < g.n_tiles; ++i)
    if (pos >= g.tile_off[i] && pos < g.tile_off[i + 1]) { t = i; break; }
  if (t < 0) return -1;
  int local = pos - g.tile_off[t];
  int r = local / g.cols[t], c = local - r * g.cols[t];
  return t * g.w * g.w + (r * g.w / g.rows[t]) * g.w + (c * g.w / g.cols[t]);
}

// ---- 16-byte vector access and element conversion -----------------------------------------------
template <typename T> struct Vec;                      // elements per 16 bytes
template <> struct Vec<__nv_bfloat16> { static constexpr int n = 8; };
template <> struct Vec<float> { static constexpr int n = 4; };

__device__ inline void unpack16(const uint4& v, float (&f)[8], __nv_bfloat16) {
  const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(u[i] << 16);
    f[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
  }
}
__device__ inline void unpack16(const uint4& v, float (&f)[4], float) {
  f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
  f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
__device__ inline uint4 pack16(const float (&f)[8], __nv_bfloat16) {
  uint32_t u[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);   // round to nearest even
    u[i] = *reinterpret_cast<uint32_t*>(&p);
  }
  return make_uint4(u[0], u[1], u[2], u[3]);
}
__device__ inline uint4 pack16(const float (&f)[4], float) {
  return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}
__device__ inline float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ inline float to_float(float v) { return v; }

// streaming 16-byte load / store (read-once data: do not keep in L1)
__device__ inline uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ inline void st_stream16(void* p, const uint4& v) {
  asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};"
               :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// monotone map float -> uint32 (ascending floats give ascending integers)
__device__ inline uint32_t orderable(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Programmatic dependent launch.  Every kernel of the library is launched with programmatic stream
// serialization and begins with this call: it lets the next kernel of the stream become resident, then
// waits until the kernel before this one has completed and its writes are visible.  So a kernel's launch
// latency hides behind its predecessor, and nothing is read or written before the predecessor is done.
// Launched without the attribute, both instructions do nothing.
__device__ __forceinline__ void grid_dependency_sync() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

}  // namespace lkv
