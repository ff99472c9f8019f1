// CRC-64 of the serialised K and V tensors (§3.4), computed while a layer is packed or
// unpacked. Reading of the paper: reflected CRC-64, all-ones initial value, final inversion,
// ISO 3309 polynomial x^64 + x^4 + x^3 + x + 1 (the paper names no polynomial).
//
// Everything is linear over GF(2). With rem(M) = M(x) * x^64 mod P (no initial value, no
// inversion) and "||" concatenation:   rem(A || B) = rem(A) * x^(8|B|) + rem(B)   (mod P).
// The tensor of one request and one plane, [layers][seq_len][kv_heads][head_dim], is cut
// into runs (a fraction of a token row); every thread owns one run: while the warp moves the
// data from source to destination it folds its run into a 64-bit remainder, multiplies that by
// x^(8 * bytes that follow the run inside its page), and the page's threads XOR their results.
// Each page then aligns its remainder inside the request's plane and XORs it into the layer's
// remainder (one atomic per page and plane); topkv_crc_finish chains the layers:
//   state_0 = ~0,  state_l+1 = state_l * x^(8 * bytes of the plane in one layer) + rem_l,
// and the checksum is ~state_L.
//
// Register convention (reflected): bit i of a 64-bit value is the coefficient of x^(63 - i);
// multiplying by x is a right shift. A little-endian 64-bit load of eight message bytes is
// their polynomial in this convention. Because the generator is sparse, x^64 = x^4+x^3+x+1
// (mod P) and a multiplication by x^64 costs a handful of shifts and XORs: no lookup table,
// pure integer ALU work (B200 has no carry-less multiply).
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "topkv_common.cuh"

namespace topkv {

constexpr uint64_t kCrcPoly = 0xD800000000000000ull;  // x^64 + x^4 + x^3 + x + 1, reflected
constexpr uint64_t kGfOne = 0x8000000000000000ull;    // the polynomial 1
constexpr uint64_t kGfX = 0x4000000000000000ull;      // the polynomial x

__host__ __device__ __forceinline__ uint64_t gf_mulx(uint64_t v) {
  return (v >> 1) ^ ((v & 1) ? kCrcPoly : 0ull);
}

// v * x^64 mod P. x^64 = x^4 + x^3 + x + 1 = (1 + x)(1 + x^3) (mod P), so two cheap steps:
// u = v + v*x, then u + u*x^3, each reduced at once. Only the top byte of the generator is
// populated, so every reduction touches the high 32-bit half only.
__host__ __device__ __forceinline__ uint64_t gf_mulx64(uint64_t v) {
  // u = v * (1 + x): the bit shifted out (degree 64) comes back as x^4 + x^3 + x + 1
  const uint64_t u = v ^ (v >> 1) ^ ((0ull - (v & 1)) & kCrcPoly);
  // u * (1 + x^3): three bits are shifted out, q = their polynomial (degree < 3, top bits);
  // q * x^64 = q * (x^4 + x^3 + x + 1) has degree < 7 and needs no further reduction
  const uint64_t q = u << 61;
  return u ^ (u >> 3) ^ q ^ (q >> 1) ^ (q >> 3) ^ (q >> 4);
}

// a * b mod P, Horner over the coefficients of a from the highest power down.
__host__ __device__ __forceinline__ uint64_t gf_mulmod(uint64_t a, uint64_t b) {
  uint64_t res = 0;
#pragma unroll 8
  for (int i = 0; i < 64; ++i) {
    res = gf_mulx(res) ^ (((a >> i) & 1) ? b : 0ull);
  }
  return res;
}

// x^n mod P by square and multiply.
__host__ __device__ inline uint64_t gf_powx(uint64_t n) {
  uint64_t result = kGfOne, base = kGfX;
  while (n) {
    if (n & 1) result = gf_mulmod(result, base);
    base = gf_mulmod(base, base);
    n >>= 1;
  }
  return result;
}

// ---- workspace (device memory owned by the caller), in 8-byte words ------------------------------
// c_run    [RB]            x^(8 * run_bytes * m)
// c_page   [maxp + 1]      x^(8 * P * row_bytes * k)
// x_req    [R]             x^(8 * s_r * row_bytes)        (per batch)
// x_last   [R]             x^(8 * v_last(r) * row_bytes)  (per batch)
// layer_rem[L * R * F]     remainder of request r, plane c in layer l: every page's CTA XORs its
//                          aligned page remainder in (atomicXor), so it starts at zero
struct CrcWorkspace {
  uint64_t* c_run;
  uint64_t* c_page;
  uint64_t* x_req;
  uint64_t* x_last;
  unsigned long long* layer_rem;
};

struct CrcGeom {
  int run_bytes;  // bytes one thread streams (divides row_bytes, multiple of 16)
  int rpr;        // runs per token row
  int RB;         // runs per page and plane = P * rpr
};

__host__ __device__ inline int64_t crc_workspace_words(int RB, int L, int R, int maxp, int F) {
  return (int64_t)RB + (maxp + 1) + 2 * (int64_t)R + (int64_t)L * R * F;
}

__host__ __device__ inline CrcWorkspace crc_carve(void* base, int RB, int L, int R, int maxp, int F) {
  (void)L;
  (void)F;
  CrcWorkspace w;
  w.c_run = static_cast<uint64_t*>(base);
  w.c_page = w.c_run + RB;
  w.x_req = w.c_page + (maxp + 1);
  w.x_last = w.x_req + R;
  w.layer_rem = reinterpret_cast<unsigned long long*>(w.x_last + R);
  return w;
}

// Builds the constant tables for this batch and clears the per-layer remainders.
__global__ void __launch_bounds__(256)
topkv_crc_begin_kernel(CrcWorkspace w, CrcGeom g, const int32_t* __restrict__ sl, int L, int R,
                       int maxp, int P, int64_t row_bytes, int F) {
  pdl_prologue(0);
  const int64_t n_run = g.RB, n_page = maxp + 1;
  const int64_t total = n_run + n_page + 2 * (int64_t)R + (int64_t)L * R * F;
  for (int64_t k = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; k < total;
       k += (int64_t)gridDim.x * blockDim.x) {
    if (k < n_run) {
      w.c_run[k] = gf_powx(8ull * g.run_bytes * (uint64_t)k);
    } else if (k < n_run + n_page) {
      const int64_t j = k - n_run;
      w.c_page[j] = gf_powx(8ull * (uint64_t)P * row_bytes * (uint64_t)j);
    } else if (k < n_run + n_page + 2 * (int64_t)R) {
      const int64_t q = k - n_run - n_page;
      const int r = (int)(q >> 1);
      int s = sl[r];
      s = max(0, min(s, maxp * P));
      const int v_last = s == 0 ? 0 : s - ((s - 1) / P) * P;
      if (q & 1) w.x_last[r] = gf_powx(8ull * (uint64_t)v_last * row_bytes);
      else w.x_req[r] = gf_powx(8ull * (uint64_t)s * row_bytes);
    } else {
      w.layer_rem[k - n_run - n_page - 2 * (int64_t)R] = 0ull;
    }
  }
}

struct CrcCopyParams {
  KParams k;
  CrcGeom g;
  CrcWorkspace w;
  int layer;
  int F;
};

constexpr int kCrcPitch = 144;          // bytes per run in the exchange tile: 128 + 16 of padding
constexpr int kCrcTileBytes = 32 * kCrcPitch;  // one tile per warp

template <int VEC>
struct Piece;
template <>
struct Piece<16> {
  uint4 a;
  __device__ __forceinline__ void load(const uint8_t* p) { a = *reinterpret_cast<const uint4*>(p); }
  __device__ __forceinline__ void store(uint8_t* p) const { *reinterpret_cast<uint4*>(p) = a; }
  __device__ __forceinline__ void to_tile(uint8_t* p) const { *reinterpret_cast<uint4*>(p) = a; }
};
template <>
struct Piece<32> {
  uint4 a, b;
  __device__ __forceinline__ void load(const uint8_t* p) {
    asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w)
                 : "l"(p));
  }
  __device__ __forceinline__ void store(uint8_t* p) const {
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(a.x), "r"(a.y),
                 "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w)
                 : "memory");
  }
  __device__ __forceinline__ void to_tile(uint8_t* p) const {
    *reinterpret_cast<uint4*>(p) = a;
    *reinterpret_cast<uint4*>(p + 16) = b;
  }
};

// One CTA per (request, page column); one thread owns one run of one plane (F * RB threads
// work). Global memory is accessed warp-coalesced: in every step the warp moves 128 bytes of
// each of several of its runs, 128 / VEC lanes per run, straight from source to destination;
// the same registers are also dropped into a padded shared-memory tile from which every lane
// picks up the 128 bytes of its OWN run, in order, for the checksum. The next batch's loads are
// issued before the current batch is folded, so that they are in flight during the ALU work.
template <int F, bool PACK, int VEC, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) topkv_crc_copy_kernel(const CrcCopyParams cp) {
  extern __shared__ __align__(16) uint8_t s_tiles[];
  __shared__ unsigned long long s_rem[2];
  constexpr int kPieces = 128 / VEC;      // pieces of one run in a batch = steps per batch
  constexpr int kRunsPerStep = 32 / kPieces;
  const KParams& p = cp.k;
  pdl_prologue(p.overlap);
  const int tid = threadIdx.x, lane = tid & 31;
  const int slot = blockIdx.x;
  const int r = slot / p.maxp;
  const int j = slot - r * p.maxp;
  int s_r = p.sl[r];
  if (s_r > p.maxp * p.P) {
    s_r = p.maxp * p.P;
    if (tid == 0 && j == 0) raise_error(kErrTable);
  }
  const int first = j * p.P;
  if (first < s_r) {
    const int v = min(p.P, s_r - first);
    const int64_t n0 = p.cu[r] + first;
    const int64_t T = p.plane_rows >= 0 ? p.plane_rows : (p.T >= 0 ? p.T : p.cu[p.R]);  // plane rows
    const int64_t row = (int64_t)cp.g.run_bytes * cp.g.rpr;
    const int64_t page = p.bt[(int64_t)r * p.maxp + j];
    const bool page_ok = page >= 0 && page < p.num_pages;
    const bool fits = p.planar ? (n0 >= 0 && ((F - 1) * T + n0 + v) * row <= p.wire_limit)
                               : (n0 >= 0 && (n0 + v) * F * row <= p.wire_limit);
    if (tid == 0 && !page_ok) raise_error(kErrTable);
    if (tid == 0 && !fits) raise_error(kErrWire);
    if (tid < 2) s_rem[tid] = 0ull;
    __syncthreads();
    const int c = tid / cp.g.RB;
    const int idx = tid - c * cp.g.RB;
    const int nruns = v * cp.g.rpr;
    const bool mine = page_ok && fits && c < F && idx < nruns;  // this lane owns a run
    // source and destination of this lane's run (null when it owns none)
    const uint8_t* src_run = nullptr;
    uint8_t* dst_run = nullptr;
    if (mine) {
      const int t = idx / cp.g.rpr;
      const int seg = idx - t * cp.g.rpr;
      uint8_t* a = p.pool + page * p.S_page + c * p.S_kv + (int64_t)t * p.S_tok +
                   (int64_t)seg * cp.g.run_bytes;
      const int64_t wrow = p.planar ? ((int64_t)c * T + n0 + t) : ((n0 + t) * F + c);
      uint8_t* b = p.wire + wrow * row + (int64_t)seg * cp.g.run_bytes;
      src_run = PACK ? a : b;
      dst_run = PACK ? b : a;
    }
    uint8_t* tile = s_tiles + (size_t)(tid >> 5) * kCrcTileBytes;
    const int sub = lane / kPieces, piece = lane % kPieces;
    uint64_t rem = 0;
    if (__any_sync(0xffffffffu, mine)) {
      // In step m this lane moves piece `piece` of the run owned by lane kRunsPerStep*m + sub.
      const uint8_t* sp[kPieces];
      uint8_t* dp[kPieces];
#pragma unroll
      for (int m = 0; m < kPieces; ++m) {
        const int owner = kRunsPerStep * m + sub;
        const uint64_t s0 = __shfl_sync(0xffffffffu, (uint64_t)src_run, owner);
        const uint64_t d0 = __shfl_sync(0xffffffffu, (uint64_t)dst_run, owner);
        sp[m] = s0 ? reinterpret_cast<const uint8_t*>(s0) + piece * VEC : nullptr;
        dp[m] = reinterpret_cast<uint8_t*>(d0) + piece * VEC;
      }
      uint8_t* my_tile_out = tile + sub * kCrcPitch + piece * VEC;  // + m * kRunsPerStep * pitch
      const uint8_t* my_tile_in = tile + lane * kCrcPitch;
      Piece<VEC> x[kPieces];
      auto fetch = [&](int off) {
        const int left = cp.g.run_bytes - off;  // bytes of every run still to move
#pragma unroll
        for (int m = 0; m < kPieces; ++m)
          if (sp[m] != nullptr && piece * VEC < left) x[m].load(sp[m] + off);
      };
      fetch(0);
      for (int off = 0; off < cp.g.run_bytes; off += 128) {
        const int left = cp.g.run_bytes - off;
#pragma unroll
        for (int m = 0; m < kPieces; ++m)
          if (sp[m] != nullptr && piece * VEC < left) {
            x[m].store(dp[m] + off);
            x[m].to_tile(my_tile_out + m * kRunsPerStep * kCrcPitch);
          }
        __syncwarp();
        if (off + 128 < cp.g.run_bytes) fetch(off + 128);  // in flight while this batch is folded
        if (mine) {
          const int words16 = min(8, left >> 4);  // never past this lane's 128 bytes of the tile
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            if (k < words16) {
              const uint4 y = *reinterpret_cast<const uint4*>(my_tile_in + k * 16);
              rem = gf_mulx64(rem ^ ((uint64_t)y.x | ((uint64_t)y.y << 32)));
              rem = gf_mulx64(rem ^ ((uint64_t)y.z | ((uint64_t)y.w << 32)));
            }
          }
        }
        __syncwarp();
      }
    }
    if (mine) {
      // align to the end of this page's plane: (nruns - 1 - idx) runs follow
      rem = gf_mulmod(rem, cp.w.c_run[nruns - 1 - idx]);
      atomicXor(&s_rem[c], (unsigned long long)rem);
    }
    __syncthreads();
    // Align this page's remainder inside the request's plane (n_r - 2 - j full pages and the
    // last, possibly partial, page follow it) and add it to the layer's remainder.
    if (tid < F && page_ok && fits) {
      const int n_r = (s_r + p.P - 1) / p.P;
      uint64_t v2 = s_rem[tid];
      if (j < n_r - 1) {
        v2 = gf_mulmod(v2, cp.w.c_page[n_r - 2 - j]);
        v2 = gf_mulmod(v2, cp.w.x_last[r]);
      }
      atomicXor(&cp.w.layer_rem[((int64_t)cp.layer * p.R + r) * F + tid], (unsigned long long)v2);
    }
  }
  pdl_epilogue(p.overlap);
}

// One thread per (request, plane): chains the layers,
//   state_0 = ~0,  state_l+1 = state_l * x^(8 * bytes of the plane in one layer) + rem_l,
// and inverts. A request without tokens has remainder 0 in every layer.
__global__ void __launch_bounds__(128)
topkv_crc_finish_kernel(CrcWorkspace w, const int32_t* __restrict__ sl, int L, int R, int F,
                        uint64_t* __restrict__ out) {
  pdl_prologue(0);
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= R * F) return;
  const int r = k / F, c = k - r * F;
  const bool empty = sl[r] <= 0;
  const uint64_t x_req = w.x_req[r];
  uint64_t state = ~0ull;
  for (int l = 0; l < L; ++l) {
    const uint64_t rem = empty ? 0ull : (uint64_t)w.layer_rem[((int64_t)l * R + r) * F + c];
    state = gf_mulmod(state, x_req) ^ rem;
  }
  out[k] = ~state;
}

}  // namespace topkv
