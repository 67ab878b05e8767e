// SOAR NVFP4 weight quantizer for NVIDIA B200 (sm_100a): kernels and the C ABI of soar.h.
//
// What runs on the device, in launch order (Algorithm 1 of the SOAR paper):
//   amax_kernel      tensor-wide max |W| and a non-finite check            (Eq. 1)
//   init_kernel      max-based scales, first codes, first tensor sums      (Eq. 1-2, Alg. 1 "Initialization")
//   iterate_kernel   T times: global scale (Eq. 5) from the previous kernel's sums, block
//                    scale (Eq. 6), candidate search (Eq. 8, App. B.3), winners stored,
//                    next sums accumulated
//   finalize_kernel  early-stop bookkeeping (Sec. 4.1), alpha and the report
//   swizzle_kernel   optional 128x4-tiled copy of the block scales
//
// State between iterations is the output itself: the packed E2M1 codes and the E4M3 scale
// bytes.  The codes that iteration t+1 starts from are the codes of iteration t's winning
// candidate (same alpha, same quantization scale), so the high-precision quantization
// scale of Sec. 3.3 never has to be stored.
//
// Arithmetic.  Whatever feeds a rounding decision is a fixed chain of IEEE binary32
// round-to-nearest operations (explicit __f*_rn intrinsics, never contracted); tensor sums
// and candidate comparisons are binary64.  Per-candidate block sums A = sum |W| m and
// B = sum m^2 are accumulated in binary32 only where that is exact (see eval_candidate).
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <mutex>
#include <vector>

#include "soar.h"

namespace {

constexpr int kThreads = 128;
constexpr size_t kWsFixedBytes = 2048;

struct Ws {
  unsigned int amax_bits;            // max over the tensor of the bf16 magnitude bit pattern
  unsigned int pad0;
  unsigned long long zero_blocks;
  unsigned long long wide;
  double sumsq;
  double num[SOAR_MAX_ITERS + 1];    // stage s: sum A_i * dd_i      (numerator of Eq. 5)
  double den[SOAR_MAX_ITERS + 1];    // stage s: sum B_i * dd_i^2    (denominator of Eq. 5)
  double sse[SOAR_MAX_ITERS + 1];    // stage s: sum of block errors (Eq. 4)
};
static_assert(sizeof(Ws) <= kWsFixedBytes, "workspace header too large");

struct Params {
  const uint16_t* W;
  uint8_t* packed;
  uint8_t* scales;     // row-major state, either the caller's buffer or workspace
  Ws* ws;
  long long ld;
  unsigned int nblk;   // rows * cols/16
  unsigned int nbc;    // cols/16
  int max_iters;
  float early_stop_rel;
  int n_dq;
  int n_beta;
  int beta_step_pct;
};

// ------------------------------------------------------------------ number formats

__device__ __forceinline__ float bits_to_mag(unsigned int bf16_bits) {
  return __uint_as_float((bf16_bits & 0x7FFFu) << 16);
}

// Value of a non-negative E4M3 code (bias 7, 3 mantissa bits, subnormals below 2^-6).
// code<<20 read as binary32 is (1+f/8)*2^(e-127) for e>0 and f*2^-129 for e==0; times 2^120
// gives (1+f/8)*2^(e-7) and f*2^-9.
__device__ __forceinline__ float e4m3_value(int code) {
  return __fmul_rn(__uint_as_float(static_cast<unsigned int>(code) << 20), 0x1p120f);
}

// Nearest E4M3 code of v >= 0 (ties to even, saturating at 448) via the sm_100a conversion.
__device__ __forceinline__ int e4m3_encode(float v) {
  unsigned short r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.0f), "f"(v));
  return r & 0xFF;
}

// Eq. 2 on a magnitude x >= 0: nearest point of {0,.5,1,1.5,2,3,4,6}, ties to the even code,
// saturating at 6.  Adding 2^(e+22), e = exponent of max(min(x,6),1), makes the binary32
// adder round to the grid step of that binade (1/2 below 2, 1 below 4, 2 above).
__device__ __forceinline__ float e2m1_round(float x) {
  float xc = fminf(x, 6.0f);
  float t = fmaxf(xc, 1.0f);
  float M = __uint_as_float((__float_as_uint(t) & 0x7F800000u) + 0x0B000000u);
  return __fsub_rn(__fadd_rn(xc, M), M);
}

// Eight grid magnitudes -> eight 4-bit codes (element 0 in the low nibble) with the sm_100a
// E2M1 conversion; the inputs are grid points, so the conversion is exact.
__device__ __forceinline__ unsigned int pack_e2m1x8(const float* m) {
  unsigned int out;
  asm("{\n"
      ".reg .b8 b0, b1, b2, b3;\n"
      "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n"
      "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n"
      "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n"
      "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n"
      "mov.b32 %0, {b0, b1, b2, b3};\n"
      "}"
      : "=r"(out)
      : "f"(m[0]), "f"(m[1]), "f"(m[2]), "f"(m[3]), "f"(m[4]), "f"(m[5]), "f"(m[6]), "f"(m[7]));
  return out;
}

// 2*magnitude of a 3-bit E2M1 code: 0,1,2,3,4,6,8,12.
__device__ __forceinline__ float e2m1_code_value(unsigned int code3) {
  const unsigned long long lut = 0x0C08060403020100ull;
  return 0.5f * static_cast<float>(static_cast<unsigned int>(lut >> (8 * code3)) & 0xFFu);
}

// ------------------------------------------------------------------ block helpers

struct Block {
  float a[16];          // magnitudes |W_j|
  unsigned int sign0;   // sign bits already at nibble bit 3 of packed word 0 / 1
  unsigned int sign1;
  float bmax;
};

__device__ __forceinline__ void load_block(const uint16_t* p, Block& blk) {
  const uint4 v0 = __ldg(reinterpret_cast<const uint4*>(p));
  const uint4 v1 = __ldg(reinterpret_cast<const uint4*>(p) + 1);
  const unsigned int w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
  unsigned int mx = 0, s0 = 0, s1 = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    blk.a[2 * i] = __uint_as_float((w[i] << 16) & 0x7FFF0000u);
    blk.a[2 * i + 1] = __uint_as_float(w[i] & 0x7FFF0000u);
    mx = __vmaxu2(mx, w[i] & 0x7FFF7FFFu);
    unsigned int sg = (((w[i] >> 15) & 1u) << 3) | ((w[i] >> 31) << 7);
    if (i < 4) s0 |= sg << (8 * i);
    else s1 |= sg << (8 * (i - 4));
  }
  blk.sign0 = s0;
  blk.sign1 = s1;
  blk.bmax = bits_to_mag(max(mx & 0xFFFFu, mx >> 16));
}

// One candidate: re-round the block under reciprocal scale r (Eq. 2) and return
// A = sum |W_j| m_j, B = sum m_j^2.  Binary32 accumulation is exact when bmax*r <= 32:
// an element with m_j > 0 then lies within 2^7 of the block maximum, every term is a
// multiple of 2^(Emin-8) and every partial sum stays below 2^24 such units.  Otherwise the
// caller switches to eval_candidate_wide.
__device__ __forceinline__ void eval_candidate(const float (&a)[16], float r, float& A, float& B) {
  float sa = 0.0f, sb = 0.0f;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    float m = e2m1_round(__fmul_rn(a[j], r));
    sa = __fmaf_rn(a[j], m, sa);
    sb = __fmaf_rn(m, m, sb);
  }
  A = sa;
  B = sb;
}

__device__ __noinline__ void eval_candidate_wide(const float (&a)[16], float r, double& A, float& B) {
  double sa = 0.0;
  float sb = 0.0f;
  for (int j = 0; j < 16; ++j) {
    float m = e2m1_round(__fmul_rn(a[j], r));
    sa = fma(static_cast<double>(a[j]), static_cast<double>(m), sa);
    sb = __fmaf_rn(m, m, sb);
  }
  A = sa;
  B = sb;
}

__device__ __forceinline__ float recip_scale(float alpha, float dq) {
  return __frcp_rn(__fmul_rn(alpha, dq));
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// Block-wide sums of up to four doubles, then one atomicAdd each from thread 0.
template <int N>
__device__ __forceinline__ void cta_accumulate(double (&v)[N], double* const (&dst)[N]) {
  __shared__ double red[N][kThreads / 32];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < N; ++i) {
    double s = warp_sum(v[i]);
    if (lane == 0) red[i][wid] = s;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int i = 0; i < N; ++i) {
      double s = 0.0;
      for (int w = 0; w < kThreads / 32; ++w) s += red[i][w];
      if (dst[i] != nullptr) atomicAdd(dst[i], s);
    }
  }
}

__device__ __forceinline__ const uint16_t* block_ptr(const Params& p, unsigned int b) {
  const unsigned int row = b / p.nbc;
  const unsigned int cb = b - row * p.nbc;
  return p.W + static_cast<long long>(row) * p.ld + static_cast<long long>(cb) * 16;
}

// Data-dependent status from the tensor maximum (bf16 magnitude bits).
__device__ __forceinline__ int status_from_amax(unsigned int amax_bits) {
  if (amax_bits >= 0x7F80u) return SOAR_STATUS_NONFINITE;
  if (amax_bits == 0) return SOAR_STATUS_ZERO_TENSOR;
  const float amax = bits_to_mag(amax_bits);
  if (!(amax >= 0x1p-100f && amax <= 0x1p100f)) return SOAR_STATUS_RANGE;
  return 0;
}

// Sec. 4.1 early stop: after an iteration, stop when the relative error gain is below eps.
__device__ __forceinline__ bool stops_after(double prev, double cur, float eps) {
  if (!(eps > 0.0f)) return false;
  if (prev == 0.0) return true;
  return (prev - cur) / prev < static_cast<double>(eps);
}

// ------------------------------------------------------------------ kernels

__global__ void __launch_bounds__(kThreads) amax_kernel(Params p) {
  unsigned int mx = 0;
  for (unsigned int b = blockIdx.x * kThreads + threadIdx.x; b < p.nblk; b += gridDim.x * kThreads) {
    const uint4* q = reinterpret_cast<const uint4*>(block_ptr(p, b));
    const uint4 v0 = __ldg(q), v1 = __ldg(q + 1);
    unsigned int m = __vmaxu2(v0.x & 0x7FFF7FFFu, v0.y & 0x7FFF7FFFu);
    m = __vmaxu2(m, v0.z & 0x7FFF7FFFu);
    m = __vmaxu2(m, v0.w & 0x7FFF7FFFu);
    m = __vmaxu2(m, v1.x & 0x7FFF7FFFu);
    m = __vmaxu2(m, v1.y & 0x7FFF7FFFu);
    m = __vmaxu2(m, v1.z & 0x7FFF7FFFu);
    m = __vmaxu2(m, v1.w & 0x7FFF7FFFu);
    mx = __vmaxu2(mx, m);
  }
  mx = max(mx & 0xFFFFu, mx >> 16);
  mx = __reduce_max_sync(0xFFFFFFFFu, mx);
  __shared__ unsigned int red[kThreads / 32];
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned int m = 0;
    for (int w = 0; w < kThreads / 32; ++w) m = max(m, red[w]);
    atomicMax(&p.ws->amax_bits, m);
  }
}

// Algorithm 1 "Initialization" (Eq. 1): alpha0 = amax/(6*448), dd0 = E4M3(bmax/(6 alpha0)),
// dq0 = dd0; first codes (Eq. 2); stage-0 sums for Eq. 5 and the starting error.
__global__ void __launch_bounds__(kThreads) init_kernel(Params p) {
  const unsigned int amax_bits = p.ws->amax_bits;
  const int st = status_from_amax(amax_bits);
  if (st & (SOAR_STATUS_NONFINITE | SOAR_STATUS_RANGE)) return;
  const float alpha = (st & SOAR_STATUS_ZERO_TENSOR) ? 1.0f : __fdiv_rn(bits_to_mag(amax_bits), 2688.0f);
  const float six_alpha = __fmul_rn(alpha, 6.0f);
  const double alpha_d = static_cast<double>(alpha);
  double acc[4] = {0.0, 0.0, 0.0, 0.0};   // num, den, sse, sumsq
  unsigned int zeros = 0;
  for (unsigned int b = blockIdx.x * kThreads + threadIdx.x; b < p.nblk; b += gridDim.x * kThreads) {
    Block blk;
    load_block(block_ptr(p, b), blk);
    uint2 out;
    if (blk.bmax == 0.0f) {
      out.x = blk.sign0;
      out.y = blk.sign1;
      reinterpret_cast<uint2*>(p.packed)[b] = out;
      p.scales[b] = 0;
      ++zeros;
      continue;
    }
    int c = e4m3_encode(__fdiv_rn(blk.bmax, six_alpha));
    c = max(c, 1);
    const float v = e4m3_value(c);
    const float r = recip_scale(alpha, v);
    float m[16];
    float Bf = 0.0f;
    double A = 0.0, S = 0.0;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      m[j] = e2m1_round(__fmul_rn(blk.a[j], r));
      const double aj = static_cast<double>(blk.a[j]);
      A = fma(aj, static_cast<double>(m[j]), A);
      S = fma(aj, aj, S);
      Bf = __fmaf_rn(m[j], m[j], Bf);
    }
    out.x = pack_e2m1x8(m) | blk.sign0;
    out.y = pack_e2m1x8(m + 8) | blk.sign1;
    reinterpret_cast<uint2*>(p.packed)[b] = out;
    p.scales[b] = static_cast<uint8_t>(c);
    const double B = static_cast<double>(Bf), vd = static_cast<double>(v);
    const double sd = alpha_d * vd;
    acc[0] += A * vd;
    acc[1] += B * vd * vd;
    acc[2] += S + sd * fma(sd, B, -2.0 * A);
    acc[3] += S;
  }
  double* const dst[4] = {&p.ws->num[0], &p.ws->den[0], &p.ws->sse[0], &p.ws->sumsq};
  cta_accumulate<4>(acc, dst);
  zeros = __reduce_add_sync(0xFFFFFFFFu, zeros);
  if ((threadIdx.x & 31) == 0 && zeros) atomicAdd(&p.ws->zero_blocks, static_cast<unsigned long long>(zeros));
}

// One iteration t of Algorithm 1 for every block: Eq. 5 (from stage-t sums), Eq. 6,
// App. B.3 candidate sets, Eq. 8 search, winner stored, stage-(t+1) sums accumulated.
__global__ void __launch_bounds__(kThreads) iterate_kernel(Params p, int t) {
  __shared__ float s_beta[SOAR_MAX_BETA];
  __shared__ float s_alpha;
  __shared__ int s_run;
  const Ws* ws = p.ws;
  if (threadIdx.x == 0) {
    int run = 1;
    const unsigned int amax_bits = ws->amax_bits;
    if (status_from_amax(amax_bits) != 0) run = 0;
    float alpha = __fdiv_rn(bits_to_mag(amax_bits), 2688.0f);
    if (run) {
      double prev = ws->sse[0];
      for (int i = 0; i < t; ++i) {           // did an earlier iteration trigger the stop?
        const double cur = ws->sse[i + 1];
        if (stops_after(prev, cur, p.early_stop_rel)) { run = 0; break; }
        prev = cur;
      }
      for (int i = 0; i <= t; ++i)            // Eq. 5: alpha^(i+1) from stage-i sums
        if (ws->den[i] > 0.0) alpha = static_cast<float>(ws->num[i] / ws->den[i]);
    }
    s_alpha = alpha;
    s_run = run;
  }
  for (int k = threadIdx.x; k < p.n_beta; k += kThreads)
    s_beta[k] = static_cast<float>((100.0 + static_cast<double>((k - p.n_beta / 2) * p.beta_step_pct)) / 100.0);
  __syncthreads();
  if (!s_run) return;
  const float alpha = s_alpha;
  const double alpha_d = static_cast<double>(alpha);
  const int n_dq = p.n_dq, n_beta = p.n_beta;

  double acc[3] = {0.0, 0.0, 0.0};   // num, den, sse of stage t+1
  unsigned int wide = 0;
  for (unsigned int b = blockIdx.x * kThreads + threadIdx.x; b < p.nblk; b += gridDim.x * kThreads) {
    const int d_cur = p.scales[b];
    if (d_cur == 0) continue;                       // all-zero block: nothing to optimise
    Block blk;
    load_block(block_ptr(p, b), blk);
    const uint2 cur = reinterpret_cast<const uint2*>(p.packed)[b];
    // Sums of the current codes (the winner of the previous stage), exact in binary64.
    double A0 = 0.0, S = 0.0;
    float B0 = 0.0f;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const unsigned int code = ((j < 8 ? cur.x : cur.y) >> (4 * (j & 7))) & 7u;
      const float m = e2m1_code_value(code);
      const double aj = static_cast<double>(blk.a[j]);
      A0 = fma(aj, static_cast<double>(m), A0);
      S = fma(aj, aj, S);
      B0 = __fmaf_rn(m, m, B0);
    }
    // Eq. 6 with the new alpha; all codes zero keeps the stored scale.
    const float center = (B0 > 0.0f)
        ? __fdiv_rn(static_cast<float>(A0), __fmul_rn(alpha, B0))
        : e4m3_value(d_cur);
    // App. B.3: E4M3 codes around the analytic scale.
    int d_lo, d_hi;
    {
      const int cn = e4m3_encode(center);
      if (n_dq <= 1) {
        d_lo = d_hi = cn;
      } else {
        const int cf = (e4m3_value(cn) > center) ? cn - 1 : cn;   // largest code with value <= center
        d_lo = cf - (n_dq / 2 - 1);
        d_hi = cf + n_dq / 2;
      }
    }
    // Eq. 8 over beta ascending, then scale code ascending; strict '<' keeps the first minimum.
    double best = __longlong_as_double(0x7FF0000000000000ll);
    double bestA = 0.0;
    float bestB = 0.0f;
    int best_k = 0, best_d = max(1, min(0x7E, d_lo));
    double prevA = -1.0;
    float prevB = -1.0f;
    for (int k = 0; k < n_beta; ++k) {
      const float r = recip_scale(alpha, __fmul_rn(center, s_beta[k]));
      double A;
      float B;
      if (__fmul_rn(blk.bmax, r) <= 32.0f) {
        float Af;
        eval_candidate(blk.a, r, Af, B);
        A = static_cast<double>(Af);
      } else {
        eval_candidate_wide(blk.a, r, A, B);
        ++wide;
      }
      if (A == prevA && B == prevB) continue;     // same sums as the previous beta: same errors
      prevA = A;
      prevB = B;
      const double Bd = static_cast<double>(B);
      for (int d = d_lo; d <= d_hi; ++d) {
        const int dc = max(1, min(0x7E, d));
        const double sd = alpha_d * static_cast<double>(e4m3_value(dc));
        const double g = sd * fma(sd, Bd, -2.0 * A);   // block error minus sum W^2
        if (g < best) { best = g; bestA = A; bestB = B; best_k = k; best_d = dc; }
      }
    }
    // Winner's codes (the assignment the next iteration, or the output, starts from).
    {
      const float r = recip_scale(alpha, __fmul_rn(center, s_beta[best_k]));
      float m[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) m[j] = e2m1_round(__fmul_rn(blk.a[j], r));
      uint2 out;
      out.x = pack_e2m1x8(m) | blk.sign0;
      out.y = pack_e2m1x8(m + 8) | blk.sign1;
      reinterpret_cast<uint2*>(p.packed)[b] = out;
      p.scales[b] = static_cast<uint8_t>(best_d);
    }
    const double vd = static_cast<double>(e4m3_value(best_d));
    acc[0] += bestA * vd;
    acc[1] += static_cast<double>(bestB) * vd * vd;
    acc[2] += S + best;
  }
  double* const dst[3] = {&p.ws->num[t + 1], &p.ws->den[t + 1], &p.ws->sse[t + 1]};
  cta_accumulate<3>(acc, dst);
  wide = __reduce_add_sync(0xFFFFFFFFu, wide);
  if ((threadIdx.x & 31) == 0 && wide) atomicAdd(&p.ws->wide, static_cast<unsigned long long>(wide));
}

// Replays the early-stop rule over the stage sums, writes alpha and the report.
__global__ void finalize_kernel(Params p, float* out_alpha, soar_result* res) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  const Ws* ws = p.ws;
  const unsigned int amax_bits = ws->amax_bits;
  const int st = status_from_amax(amax_bits);
  float alpha = (st & SOAR_STATUS_ZERO_TENSOR) ? 1.0f : __fdiv_rn(bits_to_mag(amax_bits), 2688.0f);
  int iters = 0;
  double ta[SOAR_MAX_ITERS + 1], ts[SOAR_MAX_ITERS + 1];
  ta[0] = static_cast<double>(alpha);
  ts[0] = ws->sse[0];
  if (st == 0) {
    double prev = ws->sse[0];
    for (int i = 0; i < p.max_iters; ++i) {
      if (ws->den[i] > 0.0) alpha = static_cast<float>(ws->num[i] / ws->den[i]);
      const double cur = ws->sse[i + 1];
      iters = i + 1;
      ta[iters] = static_cast<double>(alpha);
      ts[iters] = cur;
      if (stops_after(prev, cur, p.early_stop_rel)) break;
      prev = cur;
    }
  }
  *out_alpha = alpha;
  if (res != nullptr) {
    res->status = st;
    res->iters_run = iters;
    res->alpha = alpha;
    res->amax = bits_to_mag(amax_bits);
    res->sse = ts[iters];
    res->sse_init = ts[0];
    res->sumsq = ws->sumsq;
    res->zero_blocks = static_cast<int64_t>(ws->zero_blocks);
    res->wide_candidates = static_cast<int64_t>(ws->wide);
    for (int i = 0; i <= SOAR_MAX_ITERS; ++i) {
      res->trace_alpha[i] = (i <= iters) ? ta[i] : 0.0;
      res->trace_sse[i] = (i <= iters) ? ts[i] : 0.0;
    }
  }
}

// Offset of scale (row, col) in the 128x4-tiled layout: tiles of 128 rows x 4 scale columns
// (512 bytes), tile rows outermost; inside a tile row r and column c sit at
// (r % 32) * 16 + (r / 32) * 4 + c.
__device__ __forceinline__ size_t swizzled_offset(unsigned int row, unsigned int col, unsigned int col_tiles) {
  const size_t tile = static_cast<size_t>(row >> 7) * col_tiles + (col >> 2);
  const unsigned int r = row & 127u;
  return tile * 512 + (r & 31u) * 16 + (r >> 5) * 4 + (col & 3u);
}

__global__ void __launch_bounds__(256) swizzle_kernel(const uint8_t* lin, uint8_t* sw, unsigned int rows,
                                                      unsigned int nbc, unsigned int row_tiles,
                                                      unsigned int col_tiles) {
  const size_t total = static_cast<size_t>(row_tiles) * col_tiles * 512;
  for (size_t o = static_cast<size_t>(blockIdx.x) * 256 + threadIdx.x; o < total;
       o += static_cast<size_t>(gridDim.x) * 256) {
    const size_t tile = o >> 9;
    const unsigned int in = static_cast<unsigned int>(o & 511);
    const unsigned int tr = static_cast<unsigned int>(tile / col_tiles);
    const unsigned int tc = static_cast<unsigned int>(tile - static_cast<size_t>(tr) * col_tiles);
    const unsigned int row = tr * 128 + ((in >> 2) & 3u) * 32 + (in >> 4);
    const unsigned int col = tc * 4 + (in & 3u);
    sw[o] = (row < rows && col < nbc) ? lin[static_cast<size_t>(row) * nbc + col] : 0;
  }
}

// Eq. 3-4 on stored outputs.
__global__ void __launch_bounds__(kThreads) dequant_error_kernel(Params p, const uint8_t* scales, int swizzled,
                                                                 unsigned int col_tiles, const float* alpha_ptr,
                                                                 double* out_sse, double* out_sumsq) {
  const double alpha = static_cast<double>(*alpha_ptr);
  double acc[2] = {0.0, 0.0};
  for (unsigned int b = blockIdx.x * kThreads + threadIdx.x; b < p.nblk; b += gridDim.x * kThreads) {
    const unsigned int row = b / p.nbc, cb = b - row * p.nbc;
    const uint16_t* src = p.W + static_cast<long long>(row) * p.ld + static_cast<long long>(cb) * 16;
    const uint4 v0 = __ldg(reinterpret_cast<const uint4*>(src));
    const uint4 v1 = __ldg(reinterpret_cast<const uint4*>(src) + 1);
    const unsigned int w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
    const uint2 cw = reinterpret_cast<const uint2*>(p.packed)[b];
    const int dc = swizzled ? scales[swizzled_offset(row, cb, col_tiles)] : scales[b];
    const double s = alpha * static_cast<double>(e4m3_value(dc & 0x7F));
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const unsigned int word = w[j >> 1];
      const float wf = __uint_as_float((j & 1) ? (word & 0xFFFF0000u) : (word << 16));
      const unsigned int code = ((j < 8 ? cw.x : cw.y) >> (4 * (j & 7))) & 0xFu;
      const double q = static_cast<double>(e2m1_code_value(code & 7u)) * ((code & 8u) ? -1.0 : 1.0);
      const double wd = static_cast<double>(wf);
      const double e = wd - q * s;
      acc[0] = fma(e, e, acc[0]);
      acc[1] = fma(wd, wd, acc[1]);
    }
  }
  double* const dst[2] = {out_sse, out_sumsq};
  cta_accumulate<2>(acc, dst);
}

// ------------------------------------------------------------------ host side

// Optional launch tracing for benchmarks: while enabled, every kernel this library launches
// is bracketed by two CUDA events on the launching stream.
enum KernelId { K_AMAX = 0, K_INIT, K_ITERATE, K_FINALIZE, K_SWIZZLE, K_DEQUANT_ERROR, K_COUNT };
const char* const kKernelNames[K_COUNT] = {"amax_kernel",     "init_kernel",    "iterate_kernel",
                                           "finalize_kernel", "swizzle_kernel", "dequant_error_kernel"};
struct TraceRec {
  int id;
  cudaEvent_t e0, e1;
};
struct Tracer {
  std::mutex mu;
  bool on = false;
  std::vector<TraceRec> recs;
};
Tracer g_trace;

struct ScopedLaunch {
  bool active = false;
  TraceRec rec;
  cudaStream_t st;
  ScopedLaunch(int id, cudaStream_t stream) : st(stream) {
    if (!g_trace.on) return;
    rec.id = id;
    if (cudaEventCreate(&rec.e0) != cudaSuccess) return;
    if (cudaEventCreate(&rec.e1) != cudaSuccess) { cudaEventDestroy(rec.e0); return; }
    cudaEventRecord(rec.e0, st);
    active = true;
  }
  ~ScopedLaunch() {
    if (!active) return;
    cudaEventRecord(rec.e1, st);
    std::lock_guard<std::mutex> lk(g_trace.mu);
    g_trace.recs.push_back(rec);
  }
};

int g_sm_count[64];

int sm_count() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (g_sm_count[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    g_sm_count[dev] = n;
  }
  return g_sm_count[dev];
}

template <typename K>
unsigned int persistent_grid(K kernel, unsigned int nblk, int threads) {
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, 0) != cudaSuccess || per_sm <= 0)
    per_sm = 4;
  const unsigned long long cap = static_cast<unsigned long long>(sm_count()) * per_sm;
  const unsigned long long need = (static_cast<unsigned long long>(nblk) + threads - 1) / threads;
  return static_cast<unsigned int>(need < cap ? (need ? need : 1) : cap);
}

bool cfg_ok(const soar_cfg* cfg) {
  return cfg != nullptr && cfg->struct_size == sizeof(soar_cfg);
}

int check_shape(const void* W, int64_t rows, int64_t cols, int64_t ld) {
  if (W == nullptr || rows <= 0 || cols <= 0) return SOAR_ERR_INVALID_ARG;
  if (cols % 16 != 0 || ld < cols || ld % 8 != 0) return SOAR_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(W) % 16 != 0) return SOAR_ERR_UNSUPPORTED;
  if (rows * (cols / 16) >= (1ll << 31)) return SOAR_ERR_UNSUPPORTED;
  return SOAR_OK;
}

int check_cfg(const soar_cfg* cfg) {
  if (!cfg_ok(cfg)) return SOAR_ERR_INVALID_ARG;
  if (cfg->block != 16) return SOAR_ERR_UNSUPPORTED;
  if (cfg->max_iters < 0 || cfg->max_iters > SOAR_MAX_ITERS) return SOAR_ERR_INVALID_ARG;
  if (cfg->n_dq < 1 || cfg->n_dq > SOAR_MAX_DQ) return SOAR_ERR_INVALID_ARG;
  if (cfg->n_beta < 1 || cfg->n_beta > SOAR_MAX_BETA) return SOAR_ERR_INVALID_ARG;
  if (cfg->beta_step_pct < 0) return SOAR_ERR_INVALID_ARG;
  // every multiplier must stay positive
  if (100 - (cfg->n_beta / 2) * cfg->beta_step_pct <= 0) return SOAR_ERR_INVALID_ARG;
  if ((cfg->scale_layout & ~(SOAR_SCALES_LINEAR | SOAR_SCALES_SWIZZLED)) != 0 || cfg->scale_layout == 0)
    return SOAR_ERR_INVALID_ARG;
  if (cfg->flags != 0) return SOAR_ERR_INVALID_ARG;
  return SOAR_OK;
}

}  // namespace

extern "C" {

int soar_default_cfg(soar_cfg* cfg, int preset) {
  if (cfg == nullptr) return SOAR_ERR_INVALID_ARG;
  memset(cfg, 0, sizeof(*cfg));
  cfg->struct_size = sizeof(soar_cfg);
  cfg->block = 16;
  cfg->scale_layout = SOAR_SCALES_LINEAR;
  cfg->beta_step_pct = 1;
  switch (preset) {
    case SOAR_PRESET_PAPER:
      cfg->max_iters = 15; cfg->early_stop_rel = 1e-3f; cfg->n_dq = 2; cfg->n_beta = 101;
      return SOAR_OK;
    case SOAR_PRESET_SINGLE_PASS:
      cfg->max_iters = 1; cfg->early_stop_rel = 0.0f; cfg->n_dq = 2; cfg->n_beta = 1;
      return SOAR_OK;
    case SOAR_PRESET_RTN:
      cfg->max_iters = 0; cfg->early_stop_rel = 0.0f; cfg->n_dq = 1; cfg->n_beta = 1;
      return SOAR_OK;
    default:
      return SOAR_ERR_INVALID_ARG;
  }
}

size_t soar_workspace_bytes(int64_t rows, int64_t cols, const soar_cfg* cfg) {
  if (check_cfg(cfg) != SOAR_OK || rows <= 0 || cols <= 0 || cols % 16 != 0) return 0;
  size_t n = kWsFixedBytes;
  if (!(cfg->scale_layout & SOAR_SCALES_LINEAR)) {
    const size_t lin = static_cast<size_t>(rows) * static_cast<size_t>(cols / 16);
    n += (lin + 255) / 256 * 256;
  }
  return n;
}

size_t soar_swizzled_scale_bytes(int64_t rows, int64_t cols) {
  if (rows <= 0 || cols <= 0 || cols % 16 != 0) return 0;
  const size_t rt = (static_cast<size_t>(rows) + 127) / 128;
  const size_t ct = (static_cast<size_t>(cols / 16) + 3) / 4;
  return rt * ct * 512;
}

int soar_quantize_launches(const soar_cfg* cfg) {
  if (check_cfg(cfg) != SOAR_OK) return 0;
  return 3 + cfg->max_iters + ((cfg->scale_layout & SOAR_SCALES_SWIZZLED) ? 1 : 0);
}

int soar_quantize(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld, const soar_cfg* cfg,
                  void* out_fp4_packed, void* out_e4m3_scales, void* out_e4m3_scales_sw,
                  float* out_global_fp32, void* workspace, size_t workspace_bytes,
                  soar_result* out_result, void* stream) {
  int rc = check_cfg(cfg);
  if (rc != SOAR_OK) return rc;
  rc = check_shape(W_bf16, rows, cols, ld);
  if (rc != SOAR_OK) return rc;
  if (out_fp4_packed == nullptr || out_global_fp32 == nullptr) return SOAR_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(out_fp4_packed) % 16 != 0) return SOAR_ERR_UNSUPPORTED;
  const bool want_lin = (cfg->scale_layout & SOAR_SCALES_LINEAR) != 0;
  const bool want_sw = (cfg->scale_layout & SOAR_SCALES_SWIZZLED) != 0;
  if (want_lin && out_e4m3_scales == nullptr) return SOAR_ERR_INVALID_ARG;
  if (want_sw && out_e4m3_scales_sw == nullptr) return SOAR_ERR_INVALID_ARG;
  const size_t need = soar_workspace_bytes(rows, cols, cfg);
  if (workspace == nullptr || workspace_bytes < need) return SOAR_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return SOAR_ERR_UNSUPPORTED;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Params p;
  p.W = static_cast<const uint16_t*>(W_bf16);
  p.packed = static_cast<uint8_t*>(out_fp4_packed);
  p.scales = want_lin ? static_cast<uint8_t*>(out_e4m3_scales)
                      : static_cast<uint8_t*>(workspace) + kWsFixedBytes;
  p.ws = static_cast<Ws*>(workspace);
  p.ld = ld;
  p.nbc = static_cast<unsigned int>(cols / 16);
  p.nblk = static_cast<unsigned int>(rows * (cols / 16));
  p.max_iters = cfg->max_iters;
  p.early_stop_rel = cfg->early_stop_rel;
  p.n_dq = cfg->n_dq;
  p.n_beta = cfg->n_beta;
  p.beta_step_pct = cfg->beta_step_pct;

  if (cudaMemsetAsync(workspace, 0, kWsFixedBytes, st) != cudaSuccess) return SOAR_ERR_CUDA;
  {
    ScopedLaunch sl(K_AMAX, st);
    amax_kernel<<<persistent_grid(amax_kernel, p.nblk, kThreads), kThreads, 0, st>>>(p);
  }
  {
    ScopedLaunch sl(K_INIT, st);
    init_kernel<<<persistent_grid(init_kernel, p.nblk, kThreads), kThreads, 0, st>>>(p);
  }
  const unsigned int g_it = persistent_grid(iterate_kernel, p.nblk, kThreads);
  for (int t = 0; t < cfg->max_iters; ++t) {
    ScopedLaunch sl(K_ITERATE, st);
    iterate_kernel<<<g_it, kThreads, 0, st>>>(p, t);
  }
  {
    ScopedLaunch sl(K_FINALIZE, st);
    finalize_kernel<<<1, 32, 0, st>>>(p, out_global_fp32, out_result);
  }
  if (want_sw) {
    const unsigned int rt = static_cast<unsigned int>((rows + 127) / 128);
    const unsigned int ct = (p.nbc + 3) / 4;
    const size_t total = static_cast<size_t>(rt) * ct * 512;
    const size_t blocks = (total + 255) / 256;
    const unsigned int grid = static_cast<unsigned int>(blocks < 65535u * 16u ? blocks : 65535u * 16u);
    ScopedLaunch sl(K_SWIZZLE, st);
    swizzle_kernel<<<grid, 256, 0, st>>>(p.scales, static_cast<uint8_t*>(out_e4m3_scales_sw),
                                         static_cast<unsigned int>(rows), p.nbc, rt, ct);
  }
  return cudaGetLastError() == cudaSuccess ? SOAR_OK : SOAR_ERR_CUDA;
}

// Built-in scratch of soar_quantize_static.  In host code the symbol below is only a handle:
// the device address comes from cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char g_static_scratch[SOAR_STATIC_SCRATCH_BYTES];

namespace {
std::mutex g_static_mu;
void* g_static_ptr[64];

// Device address of g_static_scratch on the current device (nullptr on failure).
void* static_scratch_ptr() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lk(g_static_mu);
  if (g_static_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) return nullptr;
    g_static_ptr[dev] = ptr;
  }
  return g_static_ptr[dev];
}
}  // namespace

int soar_quantize_static(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld, const soar_cfg* cfg,
                         void* out_fp4_packed, void* out_e4m3_scales, void* out_e4m3_scales_sw,
                         float* out_global_fp32, soar_result* out_result, void* stream) {
  int rc = check_cfg(cfg);
  if (rc != SOAR_OK) return rc;
  rc = check_shape(W_bf16, rows, cols, ld);
  if (rc != SOAR_OK) return rc;
  if (rows * cols > SOAR_STATIC_MAX_ELEMENTS) return SOAR_ERR_TOO_LARGE;
  if (soar_workspace_bytes(rows, cols, cfg) > static_cast<size_t>(SOAR_STATIC_SCRATCH_BYTES))
    return SOAR_ERR_TOO_LARGE;
  void* scratch = static_scratch_ptr();
  if (scratch == nullptr) return SOAR_ERR_CUDA;
  return soar_quantize(W_bf16, rows, cols, ld, cfg, out_fp4_packed, out_e4m3_scales, out_e4m3_scales_sw,
                       out_global_fp32, scratch, SOAR_STATIC_SCRATCH_BYTES, out_result, stream);
}

int soar_dequant_error(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld, const void* fp4_packed,
                       const void* e4m3_scales, int scale_layout, const float* global_fp32,
                       double* out_sse, double* out_sumsq, void* stream) {
  const int rc = check_shape(W_bf16, rows, cols, ld);
  if (rc != SOAR_OK) return rc;
  if (fp4_packed == nullptr || e4m3_scales == nullptr || global_fp32 == nullptr || out_sse == nullptr ||
      out_sumsq == nullptr)
    return SOAR_ERR_INVALID_ARG;
  if (scale_layout != SOAR_SCALES_LINEAR && scale_layout != SOAR_SCALES_SWIZZLED) return SOAR_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(fp4_packed) % 8 != 0) return SOAR_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Params p;
  memset(&p, 0, sizeof(p));
  p.W = static_cast<const uint16_t*>(W_bf16);
  p.packed = const_cast<uint8_t*>(static_cast<const uint8_t*>(fp4_packed));
  p.ld = ld;
  p.nbc = static_cast<unsigned int>(cols / 16);
  p.nblk = static_cast<unsigned int>(rows * (cols / 16));
  if (cudaMemsetAsync(out_sse, 0, sizeof(double), st) != cudaSuccess) return SOAR_ERR_CUDA;
  if (cudaMemsetAsync(out_sumsq, 0, sizeof(double), st) != cudaSuccess) return SOAR_ERR_CUDA;
  {
    ScopedLaunch sl(K_DEQUANT_ERROR, st);
    dequant_error_kernel<<<persistent_grid(dequant_error_kernel, p.nblk, kThreads), kThreads, 0, st>>>(
        p, static_cast<const uint8_t*>(e4m3_scales), scale_layout == SOAR_SCALES_SWIZZLED ? 1 : 0,
        (p.nbc + 3) / 4, global_fp32, out_sse, out_sumsq);
  }
  return cudaGetLastError() == cudaSuccess ? SOAR_OK : SOAR_ERR_CUDA;
}

int soar_quantize_host(const void* W_host, int64_t rows, int64_t cols, int64_t ld, const soar_cfg* cfg,
                       void* out_fp4_packed_host, void* out_e4m3_scales_host, void* out_e4m3_scales_sw_host,
                       float* out_global_host, soar_result* out_result_host, const soar_staging* dev,
                       void* stream) {
  if (dev == nullptr || W_host == nullptr || dev->W == nullptr) return SOAR_ERR_INVALID_ARG;
  int rc = check_cfg(cfg);
  if (rc != SOAR_OK) return rc;
  if (rows <= 0 || cols <= 0 || ld < cols) return SOAR_ERR_INVALID_ARG;
  if (out_fp4_packed_host == nullptr || out_global_host == nullptr) return SOAR_ERR_INVALID_ARG;
  const bool want_lin = (cfg->scale_layout & SOAR_SCALES_LINEAR) != 0;
  const bool want_sw = (cfg->scale_layout & SOAR_SCALES_SWIZZLED) != 0;
  if (want_lin && (out_e4m3_scales_host == nullptr || dev->scales == nullptr)) return SOAR_ERR_INVALID_ARG;
  if (want_sw && (out_e4m3_scales_sw_host == nullptr || dev->scales_sw == nullptr)) return SOAR_ERR_INVALID_ARG;
  if (dev->packed == nullptr || dev->alpha == nullptr) return SOAR_ERR_INVALID_ARG;
  if (out_result_host != nullptr && dev->result == nullptr) return SOAR_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t in_bytes = static_cast<size_t>(rows) * static_cast<size_t>(ld) * 2;
  if (cudaMemcpyAsync(dev->W, W_host, in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return SOAR_ERR_CUDA;
  rc = soar_quantize(dev->W, rows, cols, ld, cfg, dev->packed, dev->scales, dev->scales_sw, dev->alpha,
                     dev->workspace, dev->workspace_bytes, out_result_host ? dev->result : nullptr, stream);
  if (rc != SOAR_OK) return rc;
  const size_t n = static_cast<size_t>(rows) * static_cast<size_t>(cols);
  bool ok = cudaMemcpyAsync(out_fp4_packed_host, dev->packed, n / 2, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (want_lin)
    ok = ok && cudaMemcpyAsync(out_e4m3_scales_host, dev->scales, n / 16, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (want_sw)
    ok = ok && cudaMemcpyAsync(out_e4m3_scales_sw_host, dev->scales_sw, soar_swizzled_scale_bytes(rows, cols),
                               cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(out_global_host, dev->alpha, sizeof(float), cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (out_result_host != nullptr)
    ok = ok && cudaMemcpyAsync(out_result_host, dev->result, sizeof(soar_result), cudaMemcpyDeviceToHost, st) ==
                   cudaSuccess;
  return ok ? SOAR_OK : SOAR_ERR_CUDA;
}

int soar_trace_begin(void) {
  std::lock_guard<std::mutex> lk(g_trace.mu);
  for (TraceRec& r : g_trace.recs) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
  g_trace.recs.clear();
  g_trace.on = true;
  return SOAR_OK;
}

int soar_trace_end(soar_trace_entry* out, int capacity, int* count) {
  std::lock_guard<std::mutex> lk(g_trace.mu);
  g_trace.on = false;
  double total[K_COUNT] = {0};
  int64_t launches[K_COUNT] = {0};
  bool ok = true;
  for (TraceRec& r : g_trace.recs) {
    float ms = 0.0f;
    if (cudaEventSynchronize(r.e1) != cudaSuccess || cudaEventElapsedTime(&ms, r.e0, r.e1) != cudaSuccess) ok = false;
    total[r.id] += ms;
    launches[r.id] += 1;
    cudaEventDestroy(r.e0);
    cudaEventDestroy(r.e1);
  }
  g_trace.recs.clear();
  int n = 0;
  for (int k = 0; k < K_COUNT; ++k) {
    if (launches[k] == 0) continue;
    if (out != nullptr && n < capacity) {
      memset(&out[n], 0, sizeof(out[n]));
      strncpy(out[n].kernel, kKernelNames[k], sizeof(out[n].kernel) - 1);
      out[n].launches = launches[k];
      out[n].total_ms = total[k];
    }
    ++n;
  }
  if (count != nullptr) *count = n;
  return ok ? SOAR_OK : SOAR_ERR_CUDA;
}

const char* soar_status_string(int status) {
  switch (status) {
    case SOAR_OK: return "ok";
    case SOAR_ERR_INVALID_ARG: return "invalid argument";
    case SOAR_ERR_UNSUPPORTED: return "unsupported shape, alignment or block size";
    case SOAR_ERR_WORKSPACE: return "workspace missing or too small";
    case SOAR_ERR_CUDA: return "CUDA runtime or launch error";
    case SOAR_ERR_TOO_LARGE: return "matrix exceeds the built-in scratch of soar_quantize_static";
    default: return "unknown status";
  }
}

}  // extern "C"
