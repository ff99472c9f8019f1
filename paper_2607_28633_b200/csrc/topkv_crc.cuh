// CRC-64 of the serialised K and V tensors (§3.4), computed while a layer is packed or
// unpacked. Reading of the paper: reflected CRC-64, all-ones initial value, final inversion,
// ISO 3309 polynomial x^64 + x^4 + x^3 + x + 1 (the paper names no polynomial).
//
// Everything is linear over GF(2). With rem(M) = M(x) * x^64 mod P (no initial value, no
// inversion) and "||" concatenation:   rem(A || B) = rem(A) * x^(8|B|) + rem(B)   (mod P).
// The tensor of one request and one plane, [layers][seq_len][kv_heads][head_dim], is cut,
// layer by layer, into runs (a fraction of a token row, at most 1 KiB) and the runs into
// items of 32 consecutive runs counted from the END of the request's plane, so that every item
// but the first of a request is full and k full items follow item k. One warp takes one item,
// one lane one run:
//   - the lane brings its run into its own row of the warp's shared-memory stage with one
//     bulk-async copy (cp.async.bulk, completion on the warp's mbarrier);
//   - it folds the row, 8 bytes per step, rem = (rem ^ word) * x^64, and sends the row on to
//     the destination with one bulk-async store, so no thread moves payload through registers
//     except to checksum it;
//   - it multiplies its remainder by x^(8 * run_bytes * (31 - lane)) (the runs that follow it
//     inside the item), the warp XORs the 32 results, and lane 0 stores the item's remainder.
// topkv_crc_finish multiplies item k's remainder by x^(8 * run_bytes * 32 * k), XORs the items
// of a layer, and chains the layers:
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

#include "topkv_bulk.cuh"
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

// Carry-less product of two 32-bit polynomials (bit i = coefficient of x^i here, plain order)
// with integer multipliers: each operand is split into four "every fourth bit" parts, so that
// in an integer product of two parts at most 8 terms meet in one bit position and their sum
// (< 16) cannot carry into the next position of the same class; the lowest bit of each 4-bit
// cell is then the XOR of the terms, the other three bits are masked away.
__host__ __device__ __forceinline__ uint64_t gf_clmul32(uint32_t x, uint32_t y) {
  const uint32_t x0 = x & 0x11111111u, x1 = x & 0x22222222u, x2 = x & 0x44444444u, x3 = x & 0x88888888u;
  const uint32_t y0 = y & 0x11111111u, y1 = y & 0x22222222u, y2 = y & 0x44444444u, y3 = y & 0x88888888u;
  auto m = [](uint32_t a, uint32_t b) { return (uint64_t)a * (uint64_t)b; };
  const uint64_t z0 = m(x0, y0) ^ m(x1, y3) ^ m(x2, y2) ^ m(x3, y1);
  const uint64_t z1 = m(x0, y1) ^ m(x1, y0) ^ m(x2, y3) ^ m(x3, y2);
  const uint64_t z2 = m(x0, y2) ^ m(x1, y1) ^ m(x2, y0) ^ m(x3, y3);
  const uint64_t z3 = m(x0, y3) ^ m(x1, y2) ^ m(x2, y1) ^ m(x3, y0);
  return (z0 & 0x1111111111111111ull) | (z1 & 0x2222222222222222ull) | (z2 & 0x4444444444444444ull) |
         (z3 & 0x8888888888888888ull);
}

// a * b mod P without a bit loop: a 64 x 64 carry-less product from three 32 x 32 ones
// (Karatsuba), then the reduction, which is cheap because the generator is sparse. In the
// reflected convention the plain-order product c of the two registers holds the coefficient of
// x^d in bit 126 - d: degrees 0..63 sit in bits 63..126 and degrees 64..126 in bits 62..0, so the
// low part is c >> 63, the high part (to be multiplied by x^64) is the low word shifted left once.
__host__ __device__ __forceinline__ uint64_t gf_mulmod_clmul(uint64_t a, uint64_t b) {
  const uint32_t a0 = (uint32_t)a, a1 = (uint32_t)(a >> 32), b0 = (uint32_t)b, b1 = (uint32_t)(b >> 32);
  const uint64_t lo = gf_clmul32(a0, b0), hi = gf_clmul32(a1, b1);
  const uint64_t mid = gf_clmul32(a0 ^ a1, b0 ^ b1) ^ lo ^ hi;
  const uint64_t c_lo = lo ^ (mid << 32), c_hi = hi ^ (mid >> 32);  // the 128-bit product
  return ((c_hi << 1) | (c_lo >> 63)) ^ gf_mulx64(c_lo << 1);
}

// ---- 64 message bytes per step, with the reduction put off to the end of the step -----------
// Since x^64 = m(x) = (1 + x)(1 + x^3) (mod P), eight Horner steps over the words w0..w7 give
//   new = (rem ^ w0) * m^8 + (w1 * m^6 + w2 * m^5 + ... + w6 * m + w7) * m          (mod P).
// Nothing has to be reduced on the way: a 96-bit register (three 32-bit words h:l:e, bit 95 the
// coefficient of x^0) holds every intermediate value, because each multiplication by m adds
// only 4 to the degree (63 + 7 * 4 = 91) and m^8 = 1 + x^8 + x^24 + x^32 adds 32. A
// multiplication by (1 + x^k) is "v ^= v >> k" over the three words. The 32 coefficients that
// end up in e (degrees 64..95) are brought back once per step: e(x) * x^64 = e(x) * m(x).
__host__ __device__ __forceinline__ uint32_t gf_fsr(uint32_t lo, uint32_t hi, int k) {
#ifdef __CUDA_ARCH__
  return __funnelshift_r(lo, hi, k);  // low word of (hi:lo) >> k, 0 < k < 32
#else
  return (lo >> k) | (hi << (32 - k));
#endif
}

struct Gf96 {
  uint32_t h, l, e;
};

// u * m(x) + w, unreduced (the caller keeps the degree below 96).
__host__ __device__ __forceinline__ Gf96 gf96_mulm_add(Gf96 u, uint32_t w_hi, uint32_t w_lo) {
  Gf96 a, b;  // a = u * (1 + x), b = a * (1 + x^3) + w
  a.h = u.h ^ (u.h >> 1);
  a.l = u.l ^ gf_fsr(u.l, u.h, 1);
  a.e = u.e ^ gf_fsr(u.e, u.l, 1);
  b.h = a.h ^ (a.h >> 3) ^ w_hi;
  b.l = a.l ^ gf_fsr(a.l, a.h, 3) ^ w_lo;
  b.e = a.e ^ gf_fsr(a.e, a.l, 3);
  return b;
}

// Remainder after the eight words w[0..7] (w[2i] = low half, w[2i+1] = high half of word i, as
// a little-endian load delivers them) have followed a message whose remainder was rem.
__host__ __device__ __forceinline__ uint64_t gf_fold64(uint64_t rem, const uint32_t (&w)[16]) {
  Gf96 u = {w[3], w[2], 0u};  // w1
#pragma unroll
  for (int i = 2; i < 8; ++i) u = gf96_mulm_add(u, w[2 * i + 1], w[2 * i]);
  u = gf96_mulm_add(u, 0u, 0u);  // the last * m
  const uint32_t vh = (uint32_t)(rem >> 32) ^ w[1], vl = (uint32_t)rem ^ w[0];  // rem ^ w0
  // (rem ^ w0) * (1 + x^8 + x^24 + x^32): whole-byte shifts over h:l:e
  const uint32_t h = u.h ^ vh ^ (vh >> 8) ^ (vh >> 24);
  const uint32_t l = u.l ^ vl ^ gf_fsr(vl, vh, 8) ^ gf_fsr(vl, vh, 24) ^ vh;
  const uint32_t e = u.e ^ (vl << 24) ^ (vl << 8) ^ vl;
  // e holds the coefficients of x^64 .. x^95: e * x^64 = e * (1 + x + x^3 + x^4), degree < 36
  const uint32_t rh = h ^ e ^ (e >> 1) ^ (e >> 3) ^ (e >> 4);
  const uint32_t rl = l ^ (e << 31) ^ (e << 29) ^ (e << 28);
  return ((uint64_t)rh << 32) | rl;
}

// x^n mod P, bit-serial square and multiply: the plain definition, kept as the reference that
// gf_powx is checked against on the host.
__host__ __device__ inline uint64_t gf_powx_ref(uint64_t n) {
  uint64_t result = kGfOne, base = kGfX;
  while (n) {
    if (n & 1) result = gf_mulmod(result, base);
    base = gf_mulmod(base, base);
    n >>= 1;
  }
  return result;
}

// x^n mod P, left to right over the bits of n below the leading one: square (one carry-less
// product), then one more factor x where the bit is set (a shift). About 26 products for the
// exponents met here, against several thousand dependent shift-and-add steps of the
// bit-serial form.
__host__ __device__ inline uint64_t gf_powx(uint64_t n) {
  if (n == 0) return kGfOne;
  int top = 63;
  while (!((n >> top) & 1)) --top;
  uint64_t result = kGfX;  // the leading one
  for (int b = top - 1; b >= 0; --b) {
    result = gf_mulmod_clmul(result, result);
    if ((n >> b) & 1) result = gf_mulx(result);
  }
  return result;
}

// The chain over the layers is a composition of affine maps s -> s * A + V over GF(2)[x]/P.
// then(f, g) is "f first, then g".
struct GfAffine {
  uint64_t A, V;
};
__host__ __device__ __forceinline__ GfAffine gf_then(GfAffine f, GfAffine g) {
  return {gf_mulmod_clmul(f.A, g.A), gf_mulmod_clmul(f.V, g.A) ^ g.V};
}

// ---- workspace (device memory owned by the caller), in 8-byte words ------------------------------
// c_run    [32]                 x^(8 * run_bytes * (31 - lane))
// c_tail   [kmax + 1]           x^(8 * run_bytes * 32 * k)
// x_req    [R]                  x^(8 * s_r * row_bytes)        (per batch)
// item_rem [L * R * kmax * F]   remainder of item k (counted from the end) of request r, plane c,
//                               layer l, aligned to the item's end; cleared by topkv_crc_begin,
//                               stored (not accumulated) by the copy, so packing a layer again
//                               just rewrites its entries
// layer_rem[L * R * F]          written by topkv_crc_finish
// layer_win[L] (int32)          window with which layer l was last copied (0 = all tokens), cleared
//                               by topkv_crc_begin: the chain over the layers needs every
//                               layer's own length
struct CrcWorkspace {
  uint64_t* c_run;
  uint64_t* c_tail;
  uint64_t* x_req;
  uint64_t* item_rem;
  uint64_t* layer_rem;
  int32_t* layer_win;
};

constexpr int kCrcRunsPerItem = 32;  // one run per lane
#ifndef TOPKV_CRC_RUN_MAX
#define TOPKV_CRC_RUN_MAX 1024
#endif
constexpr int kCrcRunMax = TOPKV_CRC_RUN_MAX;  // bytes one lane streams per item, at most
constexpr int kCrcMaxWarps = 16;
constexpr int kCrcMaxStages = 4;  // shared-memory stages per warp, at most
#ifndef TOPKV_CRC_STAGES
#define TOPKV_CRC_STAGES 1
#endif

struct CrcGeom {
  int run_bytes;  // bytes one lane streams per item (divides the contiguous unit, multiple of 16)
  int rpu;        // runs per contiguous unit (the whole row, or one head when heads are split)
  int rpr;        // runs per token row = units per row * rpu
  int pitch;      // bytes between the rows of a stage: odd multiple of 16 (conflict-free reads)
  int kmax;       // items per request and plane that the tables cover: ceil(maxp * P * rpr / 32)
};

__host__ __device__ inline int64_t crc_workspace_words(int kmax, int L, int R, int F) {
  return 32 + ((int64_t)kmax + 1) + (int64_t)R + (int64_t)L * R * kmax * F + (int64_t)L * R * F +
         ((int64_t)L + 1) / 2;
}

__host__ __device__ inline CrcWorkspace crc_carve(void* base, int kmax, int L, int R, int F) {
  CrcWorkspace w;
  w.c_run = static_cast<uint64_t*>(base);
  w.c_tail = w.c_run + 32;
  w.x_req = w.c_tail + (kmax + 1);
  w.item_rem = w.x_req + R;
  w.layer_rem = w.item_rem + (int64_t)L * R * kmax * F;
  w.layer_win = reinterpret_cast<int32_t*>(w.layer_rem + (int64_t)L * R * F);
  return w;
}

// Builds the constant tables for this batch and clears the item remainders.
__global__ void __launch_bounds__(256)
topkv_crc_begin_kernel(CrcWorkspace w, CrcGeom g, const int32_t* __restrict__ sl, int L, int R,
                       int maxp, int P, int64_t row_bytes, int F) {
  // No early release of the next kernel: a checksummed copy launched behind this kernel reads
  // the tables built here and writes the words cleared here, so it may only become resident
  // once every CTA of this kernel has finished.
  pdl_wait_prior_grid();
  const int64_t n_tail = (int64_t)g.kmax + 1;
  const int64_t n_items = (int64_t)L * R * g.kmax * F;
  const int64_t total = 32 + n_tail + R + n_items;
  for (int64_t k = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; k < total;
       k += (int64_t)gridDim.x * blockDim.x) {
    if (k < 32) {
      w.c_run[k] = gf_powx(8ull * g.run_bytes * (uint64_t)(31 - k));
    } else if (k < 32 + n_tail) {
      w.c_tail[k - 32] = gf_powx(8ull * g.run_bytes * 32ull * (uint64_t)(k - 32));
    } else if (k < 32 + n_tail + R) {
      const int r = (int)(k - 32 - n_tail);
      int64_t s = sl[r];
      s = s < 0 ? 0 : (s > (int64_t)maxp * P ? (int64_t)maxp * P : s);
      w.x_req[r] = gf_powx(8ull * (uint64_t)s * (uint64_t)row_bytes);
    } else {
      w.item_rem[k - 32 - n_tail - R] = 0ull;
    }
    if (k < L) w.layer_win[k] = 0;
  }
}

struct CrcCopyParams {
  KParams k;
  CrcGeom g;
  CrcWorkspace w;
  int layer;
  int stages;  // shared-memory stages per warp (1 .. kCrcMaxStages)
};

// Persistent grid; every warp runs its own pipeline of `stages` stages over the items gw,
// gw + GW, ... (gw = global warp index), so neighbouring warps work on neighbouring runs.
// Shared memory: [warps][stages] stages of 32 rows of `pitch` bytes, the mbarriers, where every
// staged run goes and which item it belongs to, the per-CTA plan
// (token prefix sums int64 [R+1] and item prefix sums int32 [R+1], rebuilt from seq_lens).
template <int F, bool PACK>
__global__ void __launch_bounds__(kCrcMaxWarps * 32, 1) topkv_crc_copy_kernel(const CrcCopyParams cp) {
  extern __shared__ __align__(128) uint8_t smem[];
  const KParams& p = cp.k;
  pdl_prologue(p.overlap);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int W = blockDim.x >> 5;
  const int run_bytes = cp.g.run_bytes, rpr = cp.g.rpr;
  const int stage_bytes = kCrcRunsPerItem * cp.g.pitch;

  const int S = cp.stages;
  uint8_t* my_row = smem + (size_t)warp * S * stage_bytes + (size_t)lane * cp.g.pitch;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)W * S * stage_bytes);
  uint8_t** s_dst = reinterpret_cast<uint8_t**>(bars + kCrcMaxWarps * kCrcMaxStages);
  int64_t* s_idx = reinterpret_cast<int64_t*>(s_dst + (size_t)W * S * 32);
  int64_t* s_cu = s_idx + (size_t)W * S;  // [R+1] tokens
  uint8_t** my_dst = s_dst + (size_t)warp * S * 32 + lane;  // [slot * 32]: where this lane's run goes
  int64_t* my_idx = s_idx + (size_t)warp * S;              // [slot]: the item's place in item_rem
  int32_t* s_ic = reinterpret_cast<int32_t*>(s_cu + (p.R + 1));     // [R+1] items per plane

  // ---- per-CTA plan ------------------------------------------------------------------------
  const int64_t row_tokens = (int64_t)p.maxp * p.P;  // what one block-table row can describe
  for (int q = threadIdx.x; q < p.R; q += blockDim.x) {
    int64_t s = p.sl[q];
    if (s < 0 || s > row_tokens) {
      raise_error(kErrTable);
      s = s < 0 ? 0 : row_tokens;
    }
    if (p.window > 0 && s > p.window) s = p.window;  // a windowed layer keeps the last min(s, W)
    s_cu[q + 1] = s;
    s_ic[q + 1] = (int32_t)((s * rpr + kCrcRunsPerItem - 1) / kCrcRunsPerItem);
  }
  if (threadIdx.x == 0) {
    s_cu[0] = 0;
    s_ic[0] = 0;
    if (blockIdx.x == 0) cp.w.layer_win[cp.layer] = p.window;  // for the chain over the layers
  }
  if (lane == 0)
    for (int q = 0; q < S; ++q) mbar_init(smem_addr(&bars[warp * kCrcMaxStages + q]), 1);
  __syncthreads();
  if (warp == 0) {  // inclusive scans, 32 entries per round
    int64_t carry_c = 0;
    int carry_i = 0;
    for (int base = 1; base <= p.R; base += 32) {
      const int q = base + lane;
      int64_t c = q <= p.R ? s_cu[q] : 0;
      int g = q <= p.R ? s_ic[q] : 0;
      for (int o = 1; o < 32; o <<= 1) {
        const int64_t c2 = __shfl_up_sync(0xffffffffu, c, o);
        const int g2 = __shfl_up_sync(0xffffffffu, g, o);
        if (lane >= o) {
          c += c2;
          g += g2;
        }
      }
      if (q <= p.R) {
        s_cu[q] = c + carry_c;
        s_ic[q] = g + carry_i;
      }
      carry_c += __shfl_sync(0xffffffffu, c, 31);
      carry_i += __shfl_sync(0xffffffffu, g, 31);
    }
  }
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  __syncthreads();

  const int64_t row = (int64_t)run_bytes * rpr;  // bytes of one [head][dim] row
  // rows from the K plane to the V plane of a PLANAR slab
  const int64_t PR = p.plane_rows >= 0 ? p.plane_rows : (p.T >= 0 ? p.T : s_cu[p.R]);
  {
    const int64_t S = s_cu[p.R];  // uniform over the grid
    const bool fits = p.planar ? ((F - 1) * PR + S) * row <= p.wire_limit : S * F * row <= p.wire_limit;
    if (!fits) {
      if (threadIdx.x == 0) raise_error(kErrWire);
      pdl_epilogue(p.overlap);
      return;
    }
  }

  const int64_t total_items = (int64_t)s_ic[p.R] * F;
  const int64_t GW = (int64_t)gridDim.x * W;
  const uint64_t c_lane = cp.w.c_run[lane];
  int64_t next_item = (int64_t)blockIdx.x * W + warp;
  bool failed = false;

  // Finds this warp's next item with anything to move. Returns false when the items are used
  // up; otherwise *src / *dst are where this lane's run comes from and goes to (null when the
  // lane has none) and *idx is the item's place in item_rem. Uniform across the warp.
  auto prepare_next = [&](const uint8_t** src_out, uint8_t** dst_out, int64_t* idx_out) -> bool {
    while (next_item < total_items) {
      const int64_t it = next_item;
      next_item += GW;
      const int m = (int)(it / F);
      const int c = (int)(it - (int64_t)m * F);
      int lo = 0, hi = p.R;  // largest r with s_ic[r] <= m
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (s_ic[mid] <= m) lo = mid;
        else hi = mid;
      }
      const int r = lo;
      const int64_t cu_r = s_cu[r];
      const int64_t kept = s_cu[r + 1] - cu_r;          // tokens this layer keeps of request r
      const int64_t n_r = kept * rpr;                   // runs of this request's plane
      const int k = s_ic[r + 1] - 1 - m;                // full items that follow this one
      const int g = (int)(n_r - (int64_t)kCrcRunsPerItem * (k + 1)) + lane;  // this lane's run
      bool active = g >= 0;
      const uint8_t* src = nullptr;
      uint8_t* dst = nullptr;
      if (active) {
        const int t = g / rpr;                               // kept token of the request
        const int u = g - t * rpr;                           // run inside the row
        const int h = u / cp.g.rpu, seg = u - h * cp.g.rpu;  // unit (head) and run inside it
        int64_t s_r = p.sl[r];                               // the kept tokens are the LAST ones
        s_r = s_r < 0 ? 0 : (s_r > row_tokens ? row_tokens : s_r);
        const int ta = (int)(s_r - kept) + t;                // token inside the sequence
        const int j = ta / p.P, tt = ta - j * p.P;
        const int64_t page = p.bt[(int64_t)r * p.maxp + j];
        if (page < 0 || page >= p.num_pages) {  // unusable entry: the run is skipped
          raise_error(kErrTable);
          active = false;
        } else {
          uint8_t* a = p.pool + page * p.S_page + c * p.S_kv + (int64_t)tt * p.S_tok +
                       (int64_t)h * p.S_unit + (int64_t)seg * run_bytes;
          const int64_t wrow = p.planar ? ((int64_t)c * PR + cu_r + t) : ((cu_r + t) * F + c);
          uint8_t* b = p.wire + wrow * row + (int64_t)u * run_bytes;
          src = PACK ? a : b;
          dst = PACK ? b : a;
        }
      }
      if (__ballot_sync(0xffffffffu, active) == 0) continue;
      *src_out = active ? src : nullptr;
      *dst_out = active ? dst : nullptr;
      *idx_out = (((int64_t)cp.layer * p.R + r) * cp.g.kmax + k) * F + c;
      return true;
    }
    return false;
  };
  // Starts the loads of a prepared item into stage `slot`: every lane brings its own run.
  auto launch_loads = [&](int slot, const uint8_t* src) {
    const unsigned mask = __ballot_sync(0xffffffffu, src != nullptr);
    const uint32_t bar = smem_addr(&bars[warp * kCrcMaxStages + slot]);
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)(__popc(mask) * run_bytes));
    __syncwarp();
    if (src != nullptr)
      bulk_g2s(smem_addr(my_row + (size_t)slot * stage_bytes), src, (uint32_t)run_bytes, bar);
  };
  auto issue_next = [&](int slot, uint8_t** dst_out, int64_t* idx_out) -> bool {
    const uint8_t* src;
    if (!prepare_next(&src, dst_out, idx_out)) return false;
    launch_loads(slot, src);
    return true;
  };

  // Sends this lane's row of stage `slot` on to `dst` and, while the store reads the row, folds
  // it; aligns the remainder to the item's end, combines the lanes, stores the item's remainder.
  auto fold_and_store = [&](int slot, uint8_t* dst, int64_t idx) {
    uint8_t* row_g = my_row + (size_t)slot * stage_bytes;
    uint64_t rem = 0;
    if (dst != nullptr) bulk_s2g(dst, smem_addr(row_g), (uint32_t)run_bytes);
    bulk_commit();
    if (dst != nullptr) {
      int off = 0;
#pragma unroll 2
      for (; off + 64 <= run_bytes; off += 64) {  // 64 bytes per step, one reduction per step
        const uint4 y0 = *reinterpret_cast<const uint4*>(row_g + off);
        const uint4 y1 = *reinterpret_cast<const uint4*>(row_g + off + 16);
        const uint4 y2 = *reinterpret_cast<const uint4*>(row_g + off + 32);
        const uint4 y3 = *reinterpret_cast<const uint4*>(row_g + off + 48);
        const uint32_t w[16] = {y0.x, y0.y, y0.z, y0.w, y1.x, y1.y, y1.z, y1.w,
                                y2.x, y2.y, y2.z, y2.w, y3.x, y3.y, y3.z, y3.w};
        rem = gf_fold64(rem, w);
      }
      for (; off < run_bytes; off += 16) {  // what is left of a run that is no multiple of 64
        const uint4 y = *reinterpret_cast<const uint4*>(row_g + off);
        rem = gf_mulx64(rem ^ ((uint64_t)y.x | ((uint64_t)y.y << 32)));
        rem = gf_mulx64(rem ^ ((uint64_t)y.z | ((uint64_t)y.w << 32)));
      }
      rem = gf_mulmod_clmul(rem, c_lane);  // 31 - lane runs follow inside the item
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) rem ^= __shfl_xor_sync(0xffffffffu, rem, o);
    if (lane == 0) cp.w.item_rem[idx] = rem;
  };
  auto wait_loaded = [&](int slot, uint32_t parity) -> bool {
    const uint32_t bar = smem_addr(&bars[warp * kCrcMaxStages + slot]);
    uint32_t polls = 0;
    while (!mbar_try_wait(bar, parity)) {
      if (++polls > kWaitPollLimit) return false;
    }
    return true;
  };

  if (S == 1) {
    // One stage per warp: load, fold, store, wait for the store to have read the rows, next item.
    // The overlap of transfers and arithmetic comes from the other warps of the SM.
    const uint8_t* src;
    uint8_t* dst;
    int64_t idx;
    uint32_t parity = 0u;
    bool have = prepare_next(&src, &dst, &idx);
    while (have) {
      launch_loads(0, src);
      uint8_t* const dst_cur = dst;
      const int64_t idx_cur = idx;
      have = prepare_next(&src, &dst, &idx);  // the next item's addresses, while the loads fly
      if (!wait_loaded(0, parity)) {
        failed = true;
        break;
      }
      parity ^= 1u;
      fold_and_store(0, dst_cur, idx_cur);
      bulk_wait_read<0>();
      __syncwarp();
    }
  } else {
    // S stages per warp. Loads run up to S - 1 items ahead. After the store of item i has been
    // issued, the stage of item i - 1 is re-filled: its store was issued one item earlier and
    // has had the whole folding of item i to read its rows out of shared memory.
    int issued = 0, consumed = 0;
    uint32_t parity_bits = 0u;  // bit q: phase parity of stage q's mbarrier
    {
      uint8_t* d;
      int64_t ix;
      while (issued < S - 1 && issue_next(issued, &d, &ix)) {
        my_dst[issued * 32] = d;
        if (lane == 0) my_idx[issued] = ix;
        ++issued;
      }
    }
    __syncwarp();
    while (consumed < issued) {
      const int cur = consumed % S;
      if (!wait_loaded(cur, (parity_bits >> cur) & 1u)) {
        failed = true;
        break;
      }
      parity_bits ^= 1u << cur;
      fold_and_store(cur, my_dst[cur * 32], my_idx[cur]);
      ++consumed;
      bulk_wait_read<1>();  // the store before the one just issued has read its rows
      __syncwarp();
      const int slot = issued % S;
      uint8_t* d;
      int64_t ix;
      if (issue_next(slot, &d, &ix)) {
        my_dst[slot * 32] = d;
        if (lane == 0) my_idx[slot] = ix;
        ++issued;
        __syncwarp();
      }
    }
  }
  if (failed && lane == 0) raise_error(kErrWait);
  bulk_wait_all();
  pdl_epilogue(p.overlap);
}

// One warp per (layer, request, plane): rem_l = XOR over the items k of item_rem * x^(8 * bytes
// that follow item k in the request's plane) = item_rem * c_tail[k].
__global__ void __launch_bounds__(128)
topkv_crc_layer_kernel(CrcWorkspace w, CrcGeom g, const int32_t* __restrict__ sl, int L, int R,
                       int F, int maxp, int P) {
  pdl_prologue(0);
  const int lane = threadIdx.x & 31;
  const int64_t q = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (q >= (int64_t)L * R * F) return;
  const int c = (int)(q % F);
  const int r = (int)((q / F) % R);
  const int l = (int)(q / ((int64_t)F * R));
  int64_t s = sl[r];
  s = s < 0 ? 0 : (s > (int64_t)maxp * P ? (int64_t)maxp * P : s);
  const int64_t win = w.layer_win[l];
  if (win > 0 && s > win) s = win;
  const int K = (int)((s * g.rpr + kCrcRunsPerItem - 1) / kCrcRunsPerItem);
  uint64_t acc = 0;
  for (int k = lane; k < K; k += 32) {
    const uint64_t v = w.item_rem[(((int64_t)l * R + r) * g.kmax + k) * F + c];
    acc ^= k == 0 ? v : gf_mulmod_clmul(v, w.c_tail[k]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) w.layer_rem[((int64_t)l * R + r) * F + c] = acc;
}

// One warp per (request, plane): chains the layers,
//   state_0 = ~0,  state_l+1 = state_l * x^(8 * bytes of the plane in layer l) + rem_l,
// and inverts. A layer copied with a window contributes min(s, window) tokens; a request
// without tokens has remainder 0 in every layer. Every step is the affine map
// s -> s * A_l + rem_l; the maps of 32 consecutive layers, one per lane, are composed by a
// shuffle tree (five levels) instead of one after the other.
__global__ void __launch_bounds__(128)
topkv_crc_finish_kernel(CrcWorkspace w, const int32_t* __restrict__ sl, int L, int R, int F, int maxp,
                        int P, int64_t row_bytes, uint64_t* __restrict__ out) {
  pdl_prologue(0);
  const int lane = threadIdx.x & 31;
  const int k = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (k >= R * F) return;  // uniform across the warp
  const int r = k / F, c = k - r * F;
  int64_t s = sl[r];
  s = s < 0 ? 0 : (s > (int64_t)maxp * P ? (int64_t)maxp * P : s);
  const uint64_t x_full = w.x_req[r];
  uint64_t x_win = 0;  // x^(8 * bytes of a windowed layer's plane), for the window this lane saw last
  int64_t seen = -1;
  uint64_t state = ~0ull;
  for (int base = 0; base < L; base += 32) {
    const int l = base + lane;
    GfAffine f = {kGfOne, 0ull};  // identity for lanes past the last layer
    if (l < L) {
      const int64_t win = w.layer_win[l];
      f.A = x_full;
      if (win > 0 && s > win) {
        if (win != seen) {
          x_win = gf_powx(8ull * (uint64_t)win * (uint64_t)row_bytes);
          seen = win;
        }
        f.A = x_win;
      }
      f.V = s == 0 ? 0ull : w.layer_rem[((int64_t)l * R + r) * F + c];
    }
    // after the step with offset o, every lane that is a multiple of 2o holds the composition of
    // the maps of lanes [lane, lane + 2o); other lanes hold values that nobody reads any more
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      GfAffine g;
      g.A = __shfl_down_sync(0xffffffffu, f.A, o);
      g.V = __shfl_down_sync(0xffffffffu, f.V, o);
      f = gf_then(f, g);
    }
    f.A = __shfl_sync(0xffffffffu, f.A, 0);
    f.V = __shfl_sync(0xffffffffu, f.V, 0);
    state = gf_mulmod_clmul(state, f.A) ^ f.V;
  }
  if (lane == 0) out[k] = ~state;
}

}  // namespace topkv
