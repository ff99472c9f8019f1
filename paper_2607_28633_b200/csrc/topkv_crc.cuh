// CRC-64 of the serialised K and V tensors (§3.4), computed while a layer is packed or
// unpacked. Reading of the paper: reflected CRC-64, all-ones initial value, final inversion,
// ISO 3309 polynomial x^64 + x^4 + x^3 + x + 1 (the paper names no polynomial).
//
// Everything is linear over GF(2). With rem(M) = M(x) * x^64 mod P (no initial value, no
// inversion) and "||" concatenation:   rem(A || B) = rem(A) * x^(8|B|) + rem(B)   (mod P).
// The tensor of one request and one plane, [layers][seq_len][kv_heads][head_dim], is cut
// into runs (a fraction of a token row); every thread streams one run through its registers on
// the way from source to destination and folds it into a 64-bit remainder, multiplies that by
// x^(8 * bytes that follow the run inside its page), and the page's threads XOR their results.
// A second, tiny kernel aligns the page remainders inside the request and chains the layers:
//   state' = state * x^(8 * bytes of this layer's plane) + rem(layer's plane),  state_0 = ~0,
// so that after the last layer the checksum is ~state.
//
// Register convention (reflected): bit i of a 64-bit value is the coefficient of x^(63 - i);
// multiplying by x is a right shift. A little-endian 64-bit load of eight message bytes is
// their polynomial in this convention. Because the generator is sparse, x^64 = x^4+x^3+x+1
// (mod P) and a multiplication by x^64 costs a handful of shifts and XORs: no table, no
// shared memory, pure integer ALU work (B200 has no carry-less multiply).
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

// v * x^64 mod P = v * (x^4 + x^3 + x + 1) mod P.
__host__ __device__ __forceinline__ uint64_t gf_mulx64(uint64_t v) {
  const uint64_t a = v ^ (v >> 1) ^ (v >> 3) ^ (v >> 4);
  // the bits shifted out have degree >= 64: q = their quotient by x^64 (degree < 4, top bits),
  // and q * x^64 = q * (x^4 + x^3 + x + 1) again, now without overflow
  const uint64_t q = (v << 63) ^ (v << 61) ^ (v << 60);
  return a ^ q ^ (q >> 1) ^ (q >> 3) ^ (q >> 4);
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

// ---- workspace (device memory owned by the caller) ---------------------------------------------
// [0]                 c_run  [max_runs]      x^(8 * run_bytes * m)
// [max_runs]          c_page [max_pages + 1] x^(8 * P * row_bytes * k)
// [.. + max_pages+1]  x_req  [R]             x^(8 * s_r * row_bytes)        (per batch)
// [.. + R]            x_last [R]             x^(8 * v_last(r) * row_bytes)  (per batch)
// [.. + R]            page_rem [R * maxp * F]
struct CrcWorkspace {
  uint64_t* c_run;
  uint64_t* c_page;
  uint64_t* x_req;
  uint64_t* x_last;
  uint64_t* page_rem;
};

struct CrcGeom {
  int run_bytes;  // bytes one thread streams (divides row_bytes, multiple of 16)
  int rpr;        // runs per token row
  int RB;         // runs per page and plane = P * rpr
};

__host__ __device__ inline CrcWorkspace crc_carve(void* base, int max_runs, int max_pages, int R) {
  CrcWorkspace w;
  w.c_run = static_cast<uint64_t*>(base);
  w.c_page = w.c_run + max_runs;
  w.x_req = w.c_page + (max_pages + 1);
  w.x_last = w.x_req + R;
  w.page_rem = w.x_last + R;
  return w;
}

// Builds the constant tables for this batch and sets every running state to ~0.
__global__ void __launch_bounds__(256)
topkv_crc_begin_kernel(CrcWorkspace w, CrcGeom g, const int32_t* __restrict__ sl, int R, int maxp,
                       int P, int64_t row_bytes, int F, uint64_t* __restrict__ state) {
  pdl_prologue(0);
  const int64_t n_run = g.RB, n_page = maxp + 1;
  const int64_t total = n_run + n_page + 2 * (int64_t)R + (int64_t)R * F;
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
      state[k - n_run - n_page - 2 * (int64_t)R] = ~0ull;
    }
  }
}

struct CrcCopyParams {
  KParams k;
  CrcGeom g;
  const uint64_t* c_run;
  uint64_t* page_rem;
};

// One CTA per (request, page column); one thread per run of one plane. F * RB threads work.
template <int F, bool PACK>
__global__ void __launch_bounds__(1024, 1) topkv_crc_copy_kernel(const CrcCopyParams cp) {
  __shared__ unsigned long long s_rem[2];
  const KParams& p = cp.k;
  pdl_prologue(p.overlap);
  const int tid = threadIdx.x;
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
    const int64_t T = p.T >= 0 ? p.T : p.cu[p.R];
    const int64_t row = (int64_t)cp.g.run_bytes * cp.g.rpr;
    const int64_t page = p.bt[(int64_t)r * p.maxp + j];
    const bool page_ok = page >= 0 && page < p.num_pages;
    const bool fits = p.planar ? (n0 >= 0 && n0 + v <= T && T * F * row <= p.wire_limit)
                               : (n0 >= 0 && (n0 + v) * F * row <= p.wire_limit);
    if (tid == 0 && !page_ok) raise_error(kErrTable);
    if (tid == 0 && !fits) raise_error(kErrWire);
    if (tid < 2) s_rem[tid] = 0ull;
    __syncthreads();
    const int c = tid / cp.g.RB;
    const int idx = tid - c * cp.g.RB;
    const int nruns = v * cp.g.rpr;
    if (page_ok && fits && c < F && idx < nruns) {
      const int t = idx / cp.g.rpr;
      const int seg = idx - t * cp.g.rpr;
      uint8_t* a = p.pool + page * p.S_page + c * p.S_kv + (int64_t)t * p.S_tok +
                   (int64_t)seg * cp.g.run_bytes;
      const int64_t wrow = p.planar ? ((int64_t)c * T + n0 + t) : ((n0 + t) * F + c);
      uint8_t* b = p.wire + wrow * row + (int64_t)seg * cp.g.run_bytes;
      const uint4* src = reinterpret_cast<const uint4*>(PACK ? a : b);
      uint4* dst = reinterpret_cast<uint4*>(PACK ? b : a);
      const int nvec = cp.g.run_bytes / 16;
      uint64_t rem = 0;
      constexpr int kBatch = 8;  // 128 bytes in flight per thread
      for (int k0 = 0; k0 < nvec; k0 += kBatch) {
        uint4 buf[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u)
          if (k0 + u < nvec) buf[u] = src[k0 + u];
#pragma unroll
        for (int u = 0; u < kBatch; ++u)
          if (k0 + u < nvec) {
            dst[k0 + u] = buf[u];
            const uint64_t w0 = (uint64_t)buf[u].x | ((uint64_t)buf[u].y << 32);
            const uint64_t w1 = (uint64_t)buf[u].z | ((uint64_t)buf[u].w << 32);
            rem = gf_mulx64(rem ^ w0);
            rem = gf_mulx64(rem ^ w1);
          }
      }
      // align to the end of this page's plane: (nruns - 1 - idx) runs follow
      rem = gf_mulmod(rem, cp.c_run[nruns - 1 - idx]);
      atomicXor(&s_rem[c], (unsigned long long)rem);
    }
    __syncthreads();
    if (tid < F) cp.page_rem[((int64_t)r * p.maxp + j) * F + tid] = page_ok && fits ? s_rem[tid] : 0ull;
  }
  pdl_epilogue(p.overlap);
}

// One CTA per (request, plane): aligns the page remainders of this layer inside the request's
// plane, XORs them, and chains the result onto the running state.
__global__ void __launch_bounds__(256)
topkv_crc_fold_kernel(CrcWorkspace w, const int32_t* __restrict__ sl, int maxp, int P, int F,
                      uint64_t* __restrict__ state) {
  __shared__ unsigned long long s_acc;
  pdl_prologue(0);
  const int r = blockIdx.x / F, c = blockIdx.x - r * F;
  int s = sl[r];
  s = max(0, min(s, maxp * P));
  const int n_r = (s + P - 1) / P;
  if (threadIdx.x == 0) s_acc = 0ull;
  __syncthreads();
  uint64_t acc = 0;
  for (int jj = threadIdx.x; jj < n_r; jj += blockDim.x) {
    uint64_t rem = w.page_rem[((int64_t)r * maxp + jj) * F + c];
    if (jj < n_r - 1) {  // followed by n_r - 2 - jj full pages and the last, possibly partial, page
      rem = gf_mulmod(rem, w.c_page[n_r - 2 - jj]);
      rem = gf_mulmod(rem, w.x_last[r]);
    }
    acc ^= rem;
  }
  for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0 && acc) atomicXor(&s_acc, (unsigned long long)acc);
  __syncthreads();
  if (threadIdx.x == 0) {
    const int64_t k = (int64_t)r * F + c;
    state[k] = gf_mulmod(state[k], w.x_req[r]) ^ s_acc;
  }
}

__global__ void topkv_crc_finish_kernel(const uint64_t* __restrict__ state, int n,
                                        uint64_t* __restrict__ out) {
  pdl_prologue(0);
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k < n) out[k] = ~state[k];
}

}  // namespace topkv
