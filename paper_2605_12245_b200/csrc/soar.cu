// SOAR NVFP4 weight quantizer for NVIDIA B200 (sm_100a): kernels and the C ABI of soar.h.
//
// What runs on the device, in launch order (Algorithm 1 of the SOAR paper):
//   amax_kernel      tensor-wide max |W|, sum W^2 and a non-finite check        (Eq. 1)
//   init_kernel      max-based scales, first codes, first tensor sums          (Eq. 1-2, Alg. 1 "Initialization")
//   iterate_kernel   T times: global scale (Eq. 5) from the previous kernel's sums, block
//                    scale (Eq. 6), candidate search (Eq. 8, App. B.3), winners stored,
//                    next sums accumulated
//   finalize_kernel  early-stop bookkeeping (Sec. 4.1), alpha and the report
//   swizzle_kernel   optional 128x4-tiled copy of the block scales
//
// Batches.  Every kernel works on up to 16 matrices at once: their tiles form one sequence
// walked by one persistent grid, so a model's many small matrices share launches; a single
// matrix is a batch of one.  Matrices that have stopped early drop out of later iterations.
//
// Data movement.  The three passes over W are persistent, warp-specialised kernels: each CTA
// walks tiles of 256 blocks (8 KB of bf16).  One thread of a producer warp fetches them with
// bulk asynchronous copies (cp.async.bulk, completion on a "full" mbarrier) into a
// four-stage shared-memory ring; 256 consumer threads, one per 16-element block, pull their
// 32 bytes into registers, hand the stage back through an "empty" mbarrier and work from
// registers, so no CTA-wide barrier sits in the tile loop and the copies of the next tiles
// are always in flight.
//
// State between iterations is 8 bytes per block in the workspace: the winner's
// A = sum |W| m (binary32, exact), 4B = sum (2m)^2 and its E4M3 scale code.  That is all
// Eq. 6 needs; the transient quantization scale of Sec. 3.3 is never stored.
//
// Arithmetic.  Whatever feeds a rounding decision is a fixed chain of IEEE binary32
// round-to-nearest operations (explicit __f*_rn intrinsics, never contracted); the E2M1
// rounding itself is the sm_100a conversion cvt.rn.satfinite.e2m1x2.f32 (nearest, ties to
// even, saturating, sign kept on zero).  Block sums A and B are integer dot products over
// 16-bit fixed-point magnitudes and the codes' byte values (dp2a / dp4a), exact whenever
// the block maximum times the reciprocal scale is at most 32; otherwise a binary64 path is
// taken.  Tensor sums and candidate comparisons are binary64.
//
// Column-weighted objective (Sec. 5 in diagonal form; soar_quantize_weighted): the same passes as
// weighted_amax_kernel, weighted_init_kernel and weighted_iterate_kernel (batched like the others).
// Block sums carry a binary32 weight per column, so they are binary64 sums in element order
// (17 bytes of state per block); the candidate loop ranks on exact integer sums over
// fixed-point images of the weighted magnitudes and falls back to binary64 sums only for
// blocks where the images' rounding could change the winner.
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#include <mutex>
#include <new>
#include <vector>

#include "soar.h"

namespace {

constexpr int kTile = 256;                     // blocks per tile = consumer threads per CTA
constexpr int kThreads = kTile + 32;           // plus one producer warp that issues the copies
constexpr int kStages = 4;                     // depth of the shared-memory ring
constexpr int kTileBytes = kTile * 32;         // 16 bf16 per block
constexpr size_t kWsFixedBytes = 2048;
constexpr unsigned int kWaitLimit = 1u << 18;  // mbarrier polls before a wait gives up (a poll takes microseconds: about a second)
constexpr unsigned int kProducerSleepNs = 32;  // the producer's pause between polls for a free stage
constexpr int kBracketMinBeta = 2;             // the bracket needs two multipliers; a single one is modes 1-3

struct Ws {
  unsigned int amax_bits;            // max over the tensor of the bf16 magnitude bit pattern
  unsigned int error;                // kErr* bits; non-zero stops the remaining passes
  unsigned long long zero_blocks;
  unsigned long long wide;
  double sumsq;                      // sum W^2
  double num[SOAR_MAX_ITERS + 1];    // stage s: sum A_i * dd_i        (numerator of Eq. 5)
  double den[SOAR_MAX_ITERS + 1];    // stage s: sum B_i * dd_i^2      (denominator of Eq. 5)
  double gsum[SOAR_MAX_ITERS + 1];   // stage s: sum of block errors minus sum W^2 (Eq. 4)
};
static_assert(sizeof(Ws) <= kWsFixedBytes, "workspace header too large");
// the same layout is published as soar_workspace_header
static_assert(kWsFixedBytes == SOAR_WORKSPACE_HEADER_BYTES && sizeof(Ws) == sizeof(soar_workspace_header) &&
                  offsetof(Ws, amax_bits) == offsetof(soar_workspace_header, amax_bits) &&
                  offsetof(Ws, error) == offsetof(soar_workspace_header, error) &&
                  offsetof(Ws, zero_blocks) == offsetof(soar_workspace_header, zero_blocks) &&
                  offsetof(Ws, wide) == offsetof(soar_workspace_header, wide) &&
                  offsetof(Ws, sumsq) == offsetof(soar_workspace_header, sumsq) &&
                  offsetof(Ws, num) == offsetof(soar_workspace_header, num) &&
                  offsetof(Ws, den) == offsetof(soar_workspace_header, den) &&
                  offsetof(Ws, gsum) == offsetof(soar_workspace_header, gsum),
              "Ws and soar_workspace_header differ");
constexpr unsigned int kErrWait = 1u;     // a bounded wait gave up
constexpr unsigned int kErrWeight = 2u;   // a column weight outside the accepted set

// Deterministic reduce mode (SOAR_FLAG_DETERMINISTIC): instead of adding its sums to the tensor's
// accumulators with atomics (in arrival order), every CTA of a pass stores them in a slot of its
// own, and the head of the next kernel adds the slots in index order.  Two stage buffers alternate
// so that a pass can fill one while late CTAs of it still read the other.
constexpr int kMaxGrid = 1024;   // no pass has more CTAs (SM count x occupancy, at most 6 per SM)
struct DetParts {
  double sumsq[kMaxGrid];          // amax pass
  double stage[2][3][kMaxGrid];    // num, den, gsum of stage s in buffer s & 1
};

struct Params {
  DetParts* det;       // per-CTA partial sums; null unless SOAR_FLAG_DETERMINISTIC
  const uint16_t* W;
  uint8_t* packed;
  uint8_t* scales;     // row-major scale bytes, either the caller's buffer or workspace
  uint2* state;        // per block {A as binary32 bits, 4B | scale code << 16}; null when T == 0
  Ws* ws;
  long long ld;
  unsigned int nblk;   // rows * cols/16
  unsigned int nbc;    // cols/16
  unsigned int ntiles;
  int contiguous;      // ld == cols: a tile is one contiguous run of bytes
  int max_iters;
  float early_stop_rel;
  int n_dq;
  int n_beta;
  int beta_step_pct;
  int flags;           // SOAR_FLAG_* bits
};

// One launch works on up to kMaxBatch tensors: their tiles form one sequence (tensor 0's tiles,
// then tensor 1's, ...), which the CTAs of the persistent grid walk together.
constexpr int kMaxBatch = 16;
struct Batch {
  int n;
  int idle_producer;          // test hook: the producer fetches nothing, so every consumer wait runs out
  unsigned int total_tiles;
  unsigned int tile_end[kMaxBatch];   // running sum of the tensors' tile counts
  Params t[kMaxBatch];
};
static_assert(sizeof(Batch) <= 3072, "kernel parameter block too large");

// What a consumer needs of its current tensor, copied out of the parameter block once per tensor.
struct Tensor {
  uint8_t* packed;
  uint8_t* scales;
  uint2* state;
  unsigned int nblk;
};
__device__ __forceinline__ Tensor tensor_view(const Params& p) {
  Tensor v;
  v.packed = p.packed;
  v.scales = p.scales;
  v.state = p.state;
  v.nblk = p.nblk;
  return v;
}

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

// Eq. 2 for eight signed values at once: nearest point of {0,.5,1,1.5,2,3,4,6} with the
// input's sign, ties to the even code, saturating at 6.  Returns eight 4-bit codes
// (sign << 3 | magnitude code), element 0 in the low nibble.
__device__ __forceinline__ unsigned int e2m1x8(float x0, float x1, float x2, float x3, float x4, float x5,
                                               float x6, float x7) {
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
      : "f"(x0), "f"(x1), "f"(x2), "f"(x3), "f"(x4), "f"(x5), "f"(x6), "f"(x7));
  return out;
}

// Four magnitude codes (the low four nibbles of `codes`, sign bits already cleared) to four
// bytes holding 2m: a byte permute over the table 0,1,2,3,4,6,8,12.
__device__ __forceinline__ unsigned int twice_magnitude_x4(unsigned int codes) {
  unsigned int out;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(out) : "r"(0x03020100u), "r"(0x0C080604u), "r"(codes));
  return out;
}

// 2*magnitude of a 3-bit E2M1 code: 0,1,2,3,4,6,8,12.
__device__ __forceinline__ float e2m1_code_value(unsigned int code3) {
  const unsigned long long lut = 0x0C08060403020100ull;
  return 0.5f * static_cast<float>(static_cast<unsigned int>(lut >> (8 * code3)) & 0xFFu);
}

// Unsigned integer to binary64 (exact).  The conversion instruction issues on the pipe of the
// special-function unit, which these kernels leave almost idle; building the value from bit
// patterns instead costs two register moves and a binary64 add on pipes that are busy
// (38.5 against 39.4 ms per Llama-3-70B-shaped layer in the candidate loop).
__device__ __forceinline__ double uint_to_double(unsigned int v) { return __uint2double_rn(v); }

// The same from bit patterns (2^52 + v, minus 2^52), for the places that convert sixteen values
// per block at once: there the conversion pipe would be the busy one.
__device__ __forceinline__ double uint_to_double_bits(unsigned int v) {
  return __hiloint2double(0x43300000, static_cast<int>(v)) - 4503599627370496.0;
}

// ------------------------------------------------------------------ shared-memory tile ring

__device__ __forceinline__ unsigned int smem_u32(const void* p) {
  return static_cast<unsigned int>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned int bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// One bulk copy global -> shared; src and dst 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned int bytes,
                                          unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// Waits for the phase with the given parity; gives up after kWaitLimit polls.  With kSleepNs > 0
// the thread sleeps that long between polls (the producer, which otherwise spins beside the
// consumer warps of its scheduler).
template <unsigned int kSleepNs = 0>
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned int parity) {
  const unsigned int addr = smem_u32(bar);
  for (unsigned int i = 0; i < kWaitLimit; ++i) {
    unsigned int ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(addr), "r"(parity)
        : "memory");
    if (ok) return true;
    if (kSleepNs > 0) __nanosleep(kSleepNs);
  }
  return false;
}

struct __align__(128) Ring {
  unsigned char tile[kStages][kTileBytes];
  unsigned long long full[kStages];    // producer -> consumers: the stage's bytes have landed
  unsigned long long empty[kStages];   // consumers -> producer: every consumer has read the stage
  int meta_tensor[kStages];            // tensor the stage's tile belongs to; -1 ends the sequence
  unsigned int meta_tile[kStages];     // and which of its tiles
  int fail;
};

// The same ring with, per stage, the tile's 8-byte block states next to its weights.
struct __align__(128) RingWithState {
  unsigned char tile[kStages][kTileBytes];
  unsigned char state[kStages][kTile * 8];
  unsigned long long full[kStages];
  unsigned long long empty[kStages];
  int meta_tensor[kStages];
  unsigned int meta_tile[kStages];
  int fail;
};

// Producer: start the copies of tile `tile` of tensor `p` into stage `s` (one copy when rows
// are contiguous, else one per row segment) and arm the stage's barrier with the byte count.
template <typename R>
__device__ __forceinline__ void ring_issue(R& ring, const Params& p, unsigned int tile, int s) {
  const unsigned int b0 = tile * kTile;
  unsigned int nb = min(static_cast<unsigned int>(kTile), p.nblk - b0);
  if constexpr (sizeof(R) == sizeof(RingWithState)) {
    // the state array is padded to 256 bytes, so rounding the copy up to 16 stays inside it
    const unsigned int sbytes = (nb * 8u + 15u) & ~15u;
    mbar_expect_tx(&ring.full[s], nb * 32u + sbytes);
    bulk_load(ring.state[s], p.state + b0, sbytes, &ring.full[s]);
  } else {
    mbar_expect_tx(&ring.full[s], nb * 32u);
  }
  unsigned char* dst = ring.tile[s];
  if (p.contiguous) {
    bulk_load(dst, p.W + static_cast<size_t>(b0) * 16, nb * 32u, &ring.full[s]);
    return;
  }
  unsigned int row = b0 / p.nbc, cb = b0 - row * p.nbc;
  while (nb > 0) {
    const unsigned int seg = min(nb, p.nbc - cb);
    bulk_load(dst, p.W + static_cast<long long>(row) * p.ld + static_cast<long long>(cb) * 16, seg * 32u,
              &ring.full[s]);
    dst += seg * 32u;
    nb -= seg;
    ++row;
    cb = 0;
  }
}

// Tensor and tile-within-tensor of position g of the batch's tile sequence.
__device__ __forceinline__ int tensor_of(const Batch& bt, unsigned int g, unsigned int& tile) {
  int ti = 0;
  unsigned int base = 0;
  while (g >= bt.tile_end[ti]) {
    base = bt.tile_end[ti];
    ++ti;
  }
  tile = g - base;
  return ti;
}

// All threads: barriers ready before anyone uses them.
template <typename R>
__device__ __forceinline__ void ring_init(R& ring) {
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&ring.full[s], 1);
      mbar_init(&ring.empty[s], kTile);
    }
    ring.fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
}

__device__ __forceinline__ bool is_producer_warp() { return threadIdx.x >= kTile; }

__device__ __forceinline__ void record_failure(const Batch& bt) {
  for (int i = 0; i < bt.n; ++i)
    if (bt.t[i].ws != nullptr) atomicOr(&bt.t[i].ws->error, kErrWait);
}

// Producer (one thread): walks the CTA's share of the tile sequence (positions blockIdx.x,
// + gridDim.x, ..., from the front or, for `reverse`, from the back: consecutive passes
// alternate so that a pass starts on what the previous one left in L2), skipping tensors
// whose bit in `run_mask` is clear, and refills a stage as soon as every consumer has handed it
// back.  After the last tile it posts an end marker.  A wait that gives up records the
// failure, lets copies still in flight land (bounded) and ends the sequence; the consumers
// then give up on their own.
template <typename R>
__device__ __forceinline__ void ring_produce(R& ring, const Batch& bt, int reverse, unsigned int run_mask) {
  if (bt.idle_producer) return;   // test hook: nothing is fetched and nothing is in flight; the consumers give up
  unsigned int n = 0;
  bool ok = true;
  for (unsigned int g0 = blockIdx.x; g0 < bt.total_tiles; g0 += gridDim.x) {
    unsigned int tile;
    const int ti = tensor_of(bt, reverse ? bt.total_tiles - 1 - g0 : g0, tile);
    if (!((run_mask >> ti) & 1u)) continue;
    const int s = static_cast<int>(n % kStages);
    if (n >= static_cast<unsigned int>(kStages)) ok = mbar_wait<kProducerSleepNs>(&ring.empty[s], (n / kStages - 1) & 1u);
    if (!ok || *static_cast<volatile int*>(&ring.fail)) { ok = false; break; }
    ring.meta_tensor[s] = ti;
    ring.meta_tile[s] = tile;
    ring_issue(ring, bt.t[ti], tile, s);
    ++n;
  }
  if (ok) {   // end marker: completes the stage's phase with no bytes
    const int s = static_cast<int>(n % kStages);
    if (n >= static_cast<unsigned int>(kStages)) ok = mbar_wait<kProducerSleepNs>(&ring.empty[s], (n / kStages - 1) & 1u);
    if (ok) {
      ring.meta_tensor[s] = -1;
      mbar_arrive(&ring.full[s]);
    }
  }
  if (!ok) {
    *static_cast<volatile int*>(&ring.fail) = 1;
    record_failure(bt);
    for (unsigned int m = (n > static_cast<unsigned int>(kStages) ? n - kStages : 0); m < n; ++m)
      (void)mbar_wait(&ring.full[m % kStages], (m / kStages) & 1u);
  }
}

// Consumer: the CTA's n-th stage.  Returns 0 with this thread's 32 bytes (and block state), the
// tile's tensor and its number, the stage handed back; 1 at the end marker; 2 when the wait
// gave up.  On 1 and 2 the caller leaves its tile loop.
template <typename R>
__device__ __forceinline__ int ring_consume(R& ring, const Batch& bt, unsigned int n, uint4& v0, uint4& v1,
                                            int& ti, unsigned int& tile, uint2* st = nullptr) {
  const int s = static_cast<int>(n % kStages);
  // the outcome is made the same for the whole warp
  if (!__all_sync(0xFFFFFFFFu, mbar_wait(&ring.full[s], (n / kStages) & 1u))) {
    *static_cast<volatile int*>(&ring.fail) = 1;
    record_failure(bt);
    return 2;
  }
  ti = ring.meta_tensor[s];
  if (ti < 0) return 1;
  tile = ring.meta_tile[s];
  const uint4* src = reinterpret_cast<const uint4*>(ring.tile[s] + threadIdx.x * 32);
  v0 = src[0];
  v1 = src[1];
  if constexpr (sizeof(R) == sizeof(RingWithState)) *st = reinterpret_cast<const uint2*>(ring.state[s])[threadIdx.x];
  mbar_arrive(&ring.empty[s]);
  return 0;
}

// ------------------------------------------------------------------ block helpers

struct Block {
  float w[16];   // the block's elements, signed
  float bmax;    // max |w_j|
};

__device__ __forceinline__ void unpack_block(const uint4& v0, const uint4& v1, Block& blk) {
  const unsigned int u[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
  float mx = 0.0f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    blk.w[2 * i] = __uint_as_float(u[i] << 16);
    blk.w[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
    mx = fmaxf(mx, fmaxf(fabsf(blk.w[2 * i]), fabsf(blk.w[2 * i + 1])));
  }
  blk.bmax = mx;
}

// Two binary32 products with one instruction (sm_100a packed multiply; each half rounds to
// nearest even exactly like a scalar multiply).
__device__ __forceinline__ void mul2(float a0, float a1, float r, float& x0, float& x1) {
  asm("{\n.reg .b64 pa, pb, pd;\n"
      "mov.b64 pa, {%2, %3};\n"
      "mov.b64 pb, {%4, %4};\n"
      "mul.rn.f32x2 pd, pa, pb;\n"
      "mov.b64 {%0, %1}, pd;\n}"
      : "=f"(x0), "=f"(x1)
      : "f"(a0), "f"(a1), "f"(r));
}

// Codes of the block under reciprocal scale r (Eq. 2): x_j = fl(w_j * r), rounded to E2M1.
__device__ __forceinline__ void round_block(const Block& blk, float r, unsigned int& c0, unsigned int& c1) {
  float x[16];
#pragma unroll
  for (int i = 0; i < 8; ++i) mul2(blk.w[2 * i], blk.w[2 * i + 1], r, x[2 * i], x[2 * i + 1]);
  c0 = e2m1x8(x[0], x[1], x[2], x[3], x[4], x[5], x[6], x[7]);
  c1 = e2m1x8(x[8], x[9], x[10], x[11], x[12], x[13], x[14], x[15]);
}

// 16-bit fixed-point magnitudes of a block: a_j = fix_j * 2^(e - 15) with 2^e <= bmax < 2^(e+1),
// exact for every element within 2^8 of the block maximum (smaller ones are rounded, and
// only ever multiplied by a zero code when bmax * r <= 32).  Two values per word.
struct Fixed {
  unsigned int pair[8];
  double unit;   // 2^(e - 16): A = unit * sum fix_j * (2 m_j)
  double inv8;   // 1 / (8 unit)
  bool ok;       // false for block maxima below 2^-110, which take the binary64 path
};

__device__ __forceinline__ void make_fixed(const Block& blk, Fixed& fx) {
  const unsigned int eb = __float_as_uint(blk.bmax) >> 23;   // biased exponent of bmax
  fx.ok = eb >= 17u;
  const unsigned int ebc = max(eb, 17u);
  const float S = __uint_as_float((269u - ebc) << 23);       // 2^(15 - e)
  fx.unit = __hiloint2double(static_cast<int>((ebc + 880u) << 20), 0);
  fx.inv8 = __hiloint2double(static_cast<int>((1163u - ebc) << 20), 0);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const unsigned int lo = __float_as_uint(__fmaf_rn(fabsf(blk.w[2 * i]), S, 8388608.0f));
    const unsigned int hi = __float_as_uint(__fmaf_rn(fabsf(blk.w[2 * i + 1]), S, 8388608.0f));
    fx.pair[i] = __byte_perm(lo, hi, 0x5410);   // low halves of lo and hi side by side
  }
}

// Integer sums of a code vector: afix = sum fix_j * (2 m_j), b4 = sum (2 m_j)^2.
__device__ __forceinline__ void code_sums(const Fixed& fx, unsigned int c0, unsigned int c1, unsigned int& afix,
                                          unsigned int& b4) {
  const unsigned int m0 = c0 & 0x77777777u, m1 = c1 & 0x77777777u;
  const unsigned int t0 = twice_magnitude_x4(m0), t1 = twice_magnitude_x4(m0 >> 16);
  const unsigned int t2 = twice_magnitude_x4(m1), t3 = twice_magnitude_x4(m1 >> 16);
  unsigned int b = __dp4a(t0, t0, 0u);
  b = __dp4a(t1, t1, b);
  b = __dp4a(t2, t2, b);
  b4 = __dp4a(t3, t3, b);
  unsigned int a = __dp2a_lo(fx.pair[0], t0, 0u);
  a = __dp2a_hi(fx.pair[1], t0, a);
  a = __dp2a_lo(fx.pair[2], t1, a);
  a = __dp2a_hi(fx.pair[3], t1, a);
  a = __dp2a_lo(fx.pair[4], t2, a);
  a = __dp2a_hi(fx.pair[5], t2, a);
  a = __dp2a_lo(fx.pair[6], t3, a);
  afix = __dp2a_hi(fx.pair[7], t3, a);
}

// The integer sums of the block's code vector under reciprocal scale r, from the magnitudes
// alone: afix = sum fix_j * (2 m_j), b4 = sum (2 m_j)^2 with m_j = E2M1(fl(a_j * r)).  Without sign
// bits the codes feed the byte permute as they are (the candidate loop only ranks; the signed
// winner is re-made later).
__device__ __forceinline__ void magnitude_sums(const float (&a)[16], const Fixed& fx, float r, unsigned int& afix,
                                               unsigned int& b4) {
  float x[16];
#pragma unroll
  for (int i = 0; i < 8; ++i) mul2(a[2 * i], a[2 * i + 1], r, x[2 * i], x[2 * i + 1]);
  const unsigned int c0 = e2m1x8(x[0], x[1], x[2], x[3], x[4], x[5], x[6], x[7]);
  const unsigned int c1 = e2m1x8(x[8], x[9], x[10], x[11], x[12], x[13], x[14], x[15]);
  const unsigned int t[4] = {twice_magnitude_x4(c0), twice_magnitude_x4(c0 >> 16), twice_magnitude_x4(c1),
                             twice_magnitude_x4(c1 >> 16)};
  unsigned int acc_a = 0, acc_b = 0;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    acc_b = __dp4a(t[q], t[q], acc_b);
    acc_a = __dp2a_lo(fx.pair[2 * q], t[q], acc_a);
    acc_a = __dp2a_hi(fx.pair[2 * q + 1], t[q], acc_a);
  }
  afix = acc_a;
  b4 = acc_b;
}

// The same sums for a code vector whose scale lies far below the block maximum: binary64
// accumulation in element order.
__device__ __forceinline__ void code_sums_wide(const float (&w)[16], unsigned int c0, unsigned int c1, double& A,
                                               double& B) {
  double sa = 0.0;
  float sb = 0.0f;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const unsigned int code = ((j < 8 ? c0 : c1) >> (4 * (j & 7))) & 7u;
    const float m = e2m1_code_value(code);
    sa = fma(static_cast<double>(fabsf(w[j])), static_cast<double>(m), sa);
    sb = __fmaf_rn(m, m, sb);
  }
  A = sa;
  B = static_cast<double>(sb);
}

// A = sum |w_j| m_j and B = sum m_j^2 of a code vector made with reciprocal scale r.
__device__ __forceinline__ void block_sums(const Block& blk, const Fixed& fx, float r, unsigned int c0,
                                           unsigned int c1, double& A, double& B, unsigned int& wide) {
  if (fx.ok && __fmul_rn(blk.bmax, r) <= 32.0f) {
    unsigned int afix, b4;
    code_sums(fx, c0, c1, afix, b4);
    A = uint_to_double(afix) * fx.unit;
    B = uint_to_double(b4) * 0.25;
  } else {
    code_sums_wide(blk.w, c0, c1, A, B);
    ++wide;
  }
}


// 1/s rounded to nearest for s in [2^-125, 2^126): the hardware's approximate reciprocal
// followed by one Newton step, y + y * (1 - s y), both as fused multiply-adds.  On sm_100a this
// equals rcp.rn for every binary32 input of that range (soar_selftest_reciprocal compares all
// of them); it is a third of the instructions.  Callers check the range (recip_fast_ok).  The
// flush-to-zero form of the approximation is used: on that range neither s nor 1/s is
// subnormal, and the plain form carries extra instructions that rescale subnormal inputs.
__device__ __forceinline__ float recip_fast(float s) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(s));
  return __fmaf_rn(y, __fmaf_rn(-s, y, 1.0f), y);
}
__device__ __forceinline__ bool recip_fast_ok(float s) {
  return ((__float_as_uint(s) >> 23) - 2u) <= 250u;   // positive, biased exponent 2 .. 252
}

// fl(1 / fl(alpha * dq)): the reciprocal scale of Eq. 2.
__device__ __forceinline__ float recip_scale(float alpha, float dq) {
  const float s = __fmul_rn(alpha, dq);
  return recip_fast_ok(s) ? recip_fast(s) : __frcp_rn(s);
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// The sixteen column weights of block column cb, widened to binary64 (exact).
__device__ __forceinline__ void load_weights(const float* h, unsigned int cb, double (&hd)[16]) {
  const float4* src = reinterpret_cast<const float4*>(h) + static_cast<size_t>(cb) * 4;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float4 v = __ldg(src + q);
    hd[4 * q] = static_cast<double>(v.x);
    hd[4 * q + 1] = static_cast<double>(v.y);
    hd[4 * q + 2] = static_cast<double>(v.z);
    hd[4 * q + 3] = static_cast<double>(v.w);
  }
}

// Per-tensor partial sums of a CTA, in shared memory.  Each consumer warp adds its sums for a
// tensor once (when the CTA's tile sequence leaves the tensor, or ends); the warp that arrives
// last forwards the CTA's total to the tensor's global accumulators, one atomicAdd each.  No
// CTA-wide barrier is involved.
template <int N, bool kDet = false>
struct Slots {
  double acc[kMaxBatch][N];
  // deterministic mode: each consumer warp's sums, added in warp order
  double part[kMaxBatch][kDet ? kTile / 32 : 1][kDet ? N : 1];
  unsigned int count[kMaxBatch];
};

// All threads, before the tile loop (a __syncthreads follows in ring_init).
template <int N, bool kDet>
__device__ __forceinline__ void slots_clear(Slots<N, kDet>& sl) {
  for (int i = threadIdx.x; i < kMaxBatch * N; i += blockDim.x) (&sl.acc[0][0])[i] = 0.0;
  for (int i = threadIdx.x; i < kMaxBatch; i += blockDim.x) sl.count[i] = 0;
}

// Whole consumer warp: adds v[] for tensor `ti` and clears it.  With `ordered` the warps' sums are kept
// apart and the last warp adds them in warp order and stores the CTA's total to dst (this CTA's own
// slot) instead of adding it to a shared accumulator: the same bits on every run.
template <int N, bool kDet>
__device__ __forceinline__ void slots_add(Slots<N, kDet>& sl, int ti, double (&v)[N], double* const (&dst)[N]) {
  constexpr bool ordered = kDet;
#pragma unroll
  for (int i = 0; i < N; ++i) v[i] = warp_sum(v[i]);
  if ((threadIdx.x & 31) == 0) {
    if (ordered) {
#pragma unroll
      for (int i = 0; i < N; ++i) sl.part[ti][threadIdx.x >> 5][i] = v[i];
    } else {
#pragma unroll
      for (int i = 0; i < N; ++i) atomicAdd(&sl.acc[ti][i], v[i]);
    }
    __threadfence_block();
    if (atomicAdd(&sl.count[ti], 1u) == kTile / 32 - 1) {
      __threadfence_block();
      if (ordered) {
#pragma unroll
        for (int i = 0; i < N; ++i) {
          double tot = 0.0;
          for (int w = 0; w < kTile / 32; ++w) tot += *static_cast<volatile double*>(&sl.part[ti][w][i]);
          *dst[i] = tot;
        }
      } else {
#pragma unroll
        for (int i = 0; i < N; ++i) atomicAdd(dst[i], atomicAdd(&sl.acc[ti][i], 0.0));
      }
    }
  }
#pragma unroll
  for (int i = 0; i < N; ++i) v[i] = 0.0;
}

// Deterministic mode, whole warp: the sum of the n per-CTA values at `parts` in a fixed order (lane l
// adds entries l, l + 32, ... in turn, then a fixed exchange tree); every lane gets the same bits.
__device__ __forceinline__ double ordered_sum(const double* parts, int n) {
  double acc = 0.0;
  for (int j = threadIdx.x & 31; j < n; j += 32) acc += parts[j];
  return warp_sum(acc);
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

// Sum of squares of a block's sixteen bf16 values in binary64 (every square is exact).  The
// widening is the float-to-double conversion instruction, which issues beside the integer pipe
// that carries the rest of the pass.
__device__ __forceinline__ void sumsq_block(const unsigned int (&u)[8], double& s0, double& s1) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const double dl = static_cast<double>(__uint_as_float(u[i] << 16));
    const double dh = static_cast<double>(__uint_as_float(u[i] & 0xFFFF0000u));
    s0 = fma(dl, dl, s0);
    s1 = fma(dh, dh, s1);
  }
}

// Eq. 1's tensor maximum, plus sum W^2 (binary64) for the error report.
template <bool kDet>
__global__ void __launch_bounds__(kThreads, 6) amax_kernel(const __grid_constant__ Batch bt, int reverse) {
  __shared__ Ring ring;
  __shared__ Slots<1, kDet> slots;
  slots_clear(slots);
  constexpr bool det = kDet;
  if (det && threadIdx.x < bt.n) bt.t[threadIdx.x].det->sumsq[blockIdx.x] = 0.0;   // a CTA may never meet a tensor
  ring_init(ring);
  if (is_producer_warp()) {
    if (threadIdx.x == kTile) ring_produce(ring, bt, reverse, 0xFFFFFFFFu);
    return;
  }
  unsigned int mx = 0, nblk = 0;
  double sq[2] = {0.0, 0.0};
  int cur = -1;
  for (unsigned int n = 0;; ++n) {
    uint4 v0, v1;
    int ti = -1;
    unsigned int tile = 0;
    const int rc = ring_consume(ring, bt, n, v0, v1, ti, tile);
    if (rc != 0 || ti != cur) {
      if (cur >= 0) {   // leaving tensor `cur`: hand over its maximum and sum
        mx = max(mx & 0xFFFFu, mx >> 16);
        mx = __reduce_max_sync(0xFFFFFFFFu, mx);
        if ((threadIdx.x & 31) == 0 && mx) atomicMax(&bt.t[cur].ws->amax_bits, mx);
        double acc[1] = {sq[0] + sq[1]};
        double* const dst[1] = {det ? &bt.t[cur].det->sumsq[blockIdx.x] : &bt.t[cur].ws->sumsq};
        slots_add(slots, cur, acc, dst);
        mx = 0;
        sq[0] = sq[1] = 0.0;
      }
      if (rc != 0) break;
      cur = ti;
      nblk = bt.t[ti].nblk;
    }
    if (tile * kTile + threadIdx.x >= nblk) continue;
    const unsigned int u[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
    // largest magnitude of the block with packed bf16 max (a NaN input comes out of the maximum
    // as NaN, whose bits are above the infinity pattern)
    unsigned int bmx = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      unsigned int m;
      asm("abs.bf16x2 %0, %1;" : "=r"(m) : "r"(u[i]));
      asm("max.NaN.bf16x2 %0, %0, %1;" : "+r"(bmx) : "r"(m));
    }
    bmx &= 0x7FFF7FFFu;
    mx = __vmaxu2(mx, bmx);
    sumsq_block(u, sq[0], sq[1]);
  }
}

// Warp-level hand-over of two counters to a tensor's workspace.
__device__ __forceinline__ void add_counters(Ws* ws, unsigned int& zeros, unsigned int& wide) {
  zeros = __reduce_add_sync(0xFFFFFFFFu, zeros);
  wide = __reduce_add_sync(0xFFFFFFFFu, wide);
  if ((threadIdx.x & 31) == 0) {
    if (zeros) atomicAdd(&ws->zero_blocks, static_cast<unsigned long long>(zeros));
    if (wide) atomicAdd(&ws->wide, static_cast<unsigned long long>(wide));
  }
  zeros = wide = 0;
}

// Algorithm 1 "Initialization" (Eq. 1): alpha0 = amax/(6*448), dd0 = E4M3(bmax/(6 alpha0)),
// dq0 = dd0; first codes (Eq. 2); stage-0 sums for Eq. 5 and the starting error.  Codes and
// scales are written here only when no iteration follows (final != 0).  Tensors with
// non-finite or out-of-range input are skipped.
template <bool kDet>
__global__ void __launch_bounds__(kThreads) init_kernel(const __grid_constant__ Batch bt, int reverse, int final,
                                                        int prev_grid) {
  __shared__ Ring ring;
  __shared__ Slots<3, kDet> slots;
  slots_clear(slots);
  constexpr bool det = kDet;
  if (det) {
    // this CTA's stage-0 slots start at zero; CTA 0 adds up the amax pass's per-CTA sums of squares in order
    for (int i = threadIdx.x; i < bt.n * 3; i += kThreads) bt.t[i / 3].det->stage[0][i % 3][blockIdx.x] = 0.0;
    if (blockIdx.x == 0)
      for (int ti = threadIdx.x >> 5; ti < bt.n; ti += kThreads / 32) {
        const double sq = ordered_sum(bt.t[ti].det->sumsq, prev_grid);
        if ((threadIdx.x & 31) == 0) bt.t[ti].ws->sumsq = sq;
      }
  }
  ring_init(ring);
  if (is_producer_warp()) {
    if (threadIdx.x == kTile) {
      unsigned int run = 0;
      for (int i = 0; i < bt.n; ++i)
        if (!(status_from_amax(bt.t[i].ws->amax_bits) & (SOAR_STATUS_NONFINITE | SOAR_STATUS_RANGE))) run |= 1u << i;
      ring_produce(ring, bt, reverse, run);
    }
    return;
  }
  float alpha = 1.0f, six_alpha = 6.0f;
  double alpha_d = 1.0;
  double acc[3] = {0.0, 0.0, 0.0};   // num, den, gsum
  unsigned int zeros = 0, wide = 0;
  int cur = -1;
  Tensor p = {};   // the current tensor's pointers and size, kept in registers
  for (unsigned int n = 0;; ++n) {
    uint4 v0, v1;
    int ti = -1;
    unsigned int tile = 0;
    const int rc = ring_consume(ring, bt, n, v0, v1, ti, tile);
    if (rc != 0 || ti != cur) {
      if (cur >= 0) {
        Ws* ws = bt.t[cur].ws;
        DetParts* dp = bt.t[cur].det;
        double* const dst[3] = {det ? &dp->stage[0][0][blockIdx.x] : &ws->num[0],
                                det ? &dp->stage[0][1][blockIdx.x] : &ws->den[0],
                                det ? &dp->stage[0][2][blockIdx.x] : &ws->gsum[0]};
        slots_add(slots, cur, acc, dst);
        add_counters(ws, zeros, wide);
      }
      if (rc != 0) break;
      cur = ti;
      const unsigned int amax_bits = bt.t[ti].ws->amax_bits;
      alpha = amax_bits == 0 ? 1.0f : __fdiv_rn(bits_to_mag(amax_bits), 2688.0f);
      six_alpha = __fmul_rn(alpha, 6.0f);
      alpha_d = static_cast<double>(alpha);
      p = tensor_view(bt.t[ti]);
    }
    const unsigned int b = tile * kTile + threadIdx.x;
    if (b >= p.nblk) continue;
    Block blk;
    unpack_block(v0, v1, blk);
    uint2 codes;
    if (blk.bmax == 0.0f) {
      // all-zero block: codes carry the sign bits only, scale byte 0, left out of all sums
      round_block(blk, 1.0f, codes.x, codes.y);
      reinterpret_cast<uint2*>(p.packed)[b] = codes;
      p.scales[b] = 0;
      if (p.state != nullptr) p.state[b] = make_uint2(0u, 0u);
      ++zeros;
      continue;
    }
    int c = e4m3_encode(__fdiv_rn(blk.bmax, six_alpha));
    c = max(c, 1);
    const float v = e4m3_value(c);
    const float r = recip_scale(alpha, v);
    round_block(blk, r, codes.x, codes.y);
    Fixed fx;
    make_fixed(blk, fx);
    double A, B;
    block_sums(blk, fx, r, codes.x, codes.y, A, B, wide);
    if (final) {
      reinterpret_cast<uint2*>(p.packed)[b] = codes;
      p.scales[b] = static_cast<uint8_t>(c);
    }
    if (p.state != nullptr)
      p.state[b] = make_uint2(__float_as_uint(static_cast<float>(A)),
                              static_cast<unsigned int>(B * 4.0) | (static_cast<unsigned int>(c) << 16));
    const double vd = static_cast<double>(v);
    const double sd = alpha_d * vd;
    acc[0] = fma(A, vd, acc[0]);
    acc[1] = fma(B * vd, vd, acc[1]);
    acc[2] += sd * fma(sd, B, -2.0 * A);
  }
}

// Error of stage s (Eq. 4) from the tensor sums.
__device__ __forceinline__ double stage_sse(const Ws* ws, int s) {
  return fmax(ws->sumsq + ws->gsum[s], 0.0);
}

// Head of an iteration (one thread): has the loop already stopped (Sec. 4.1), and the global
// scale of Eq. 5 from the sums of the stages so far.
// `latest` (deterministic mode): num, den, gsum of stage t, which the workspace does not hold yet.
__device__ __forceinline__ void iteration_head(const Params& p, int t, float& alpha_out, int& run_out,
                                               const double* latest = nullptr) {
  const Ws* ws = p.ws;
  int run = 1;
  const unsigned int amax_bits = ws->amax_bits;
  if (status_from_amax(amax_bits) != 0 || ws->error != 0) run = 0;
  float alpha = __fdiv_rn(bits_to_mag(amax_bits), 2688.0f);
  if (run) {
    double prev = stage_sse(ws, 0);
    if (latest != nullptr && t == 0) prev = fmax(ws->sumsq + latest[2], 0.0);
    for (int i = 0; i < t; ++i) {           // did an earlier iteration trigger the stop?
      const double cur = (latest != nullptr && i + 1 == t) ? fmax(ws->sumsq + latest[2], 0.0) : stage_sse(ws, i + 1);
      if (stops_after(prev, cur, p.early_stop_rel)) { run = 0; break; }
      prev = cur;
    }
    if (!(p.flags & SOAR_FLAG_KEEP_ALPHA))
      for (int i = 0; i <= t; ++i) {        // Eq. 5: alpha^(i+1) from stage-i sums
        const double num = (latest != nullptr && i == t) ? latest[0] : ws->num[i];
        const double den = (latest != nullptr && i == t) ? latest[1] : ws->den[i];
        if (den > 0.0) alpha = static_cast<float>(num / den);
      }
  }
  alpha_out = alpha;
  run_out = run;
}

// Deterministic mode, head of the kernel that follows the pass which filled stage s (iteration s, or
// the last kernel of the call): whole CTA.  For every tensor whose stage-s slots are current (the
// filling pass worked on it), the slots of the `prev_grid` CTAs are added in index order into
// latest[tensor][0..2]; CTA 0 also files the sums in the workspace header, where later kernels
// read the stages before their own.  Every CTA computes the same bits.
__device__ __forceinline__ void gather_stage(const Batch& bt, int s, int prev_grid, double (*latest)[3]) {
  for (int ti = threadIdx.x >> 5; ti < bt.n; ti += blockDim.x >> 5) {
    const Params& p = bt.t[ti];
    int filled = 1;   // stage 0 comes from the init pass, which fills every tensor's slots
    if (s > 0) {
      float unused;
      iteration_head(p, s - 1, unused, filled);
    }
    double v[3] = {0.0, 0.0, 0.0};
    if (filled) {
#pragma unroll
      for (int i = 0; i < 3; ++i) v[i] = ordered_sum(p.det->stage[s & 1][i], prev_grid);
    }
    if ((threadIdx.x & 31) == 0) {
#pragma unroll
      for (int i = 0; i < 3; ++i) latest[ti][i] = v[i];
      if (filled && blockIdx.x == 0) {
        p.ws->num[s] = v[0];
        p.ws->den[s] = v[1];
        p.ws->gsum[s] = v[2];
      }
    }
  }
}

// App. B.3's E4M3 codes around a block's analytic scale: d_lo .. d_hi before clipping (the
// nearest code alone for n_dq == 1, else n_dq codes bracketing the scale).
__device__ __forceinline__ void candidate_window(float center, int n_dq, int& d_lo, int& d_hi) {
  const int cn = e4m3_encode(center);
  if (n_dq <= 1) {
    d_lo = d_hi = cn;
  } else {
    const int cf = (e4m3_value(cn) > center) ? cn - 1 : cn;   // largest code with value <= center
    d_lo = cf - (n_dq / 2 - 1);
    d_hi = cf + n_dq / 2;
  }
}

// Eq. 6 with the new alpha from the previous winner's sums (all codes zero keeps the stored
// scale), and the candidate codes around it.
__device__ __forceinline__ float block_center(const uint2 st, float alpha, int n_dq, bool keep, int& d_lo,
                                              int& d_hi) {
  const int d_cur = static_cast<int>(st.y >> 16);
  const float B0 = 0.25f * static_cast<float>(st.y & 0xFFFFu);
  const float center = (B0 > 0.0f && !keep) ? __fdiv_rn(__uint_as_float(st.x), __fmul_rn(alpha, B0))
                                             : e4m3_value(d_cur);
  candidate_window(center, n_dq, d_lo, d_hi);
  return center;
}

__device__ __forceinline__ int clip_code(int d) { return max(1, min(0x7E, d)); }

// fl(alpha * fl(center * beta)): the divisor of Eq. 2 for one multiplier of the App. B.3 grid.
__device__ __forceinline__ float grid_divisor(float alpha, float center, float beta) {
  return __fmul_rn(alpha, __fmul_rn(center, beta));
}

// Which multipliers of the App. B.3 grid can win Eq. 8 for one E4M3 code, without visiting the grid.
//
// For a fixed dequantization scale sd = alpha * value(code) the error of element j,
// (a_j - m sd)^2, is convex in its code value m with its minimum at a_j / sd.  The codes
// m_j(k) = E2M1(fl(a_j * fl(1 / s_k))), s_k = grid_divisor(beta_k), never rise with k, because every
// step of that binary32 chain is monotone.  While s_k <= sd (1 - 2^-21) every fl(a_j * fl(1 / s_k)) lies
// above a_j / sd (by at least 2^-22 of it: the chain's two roundings cost 2^-24 each), so every code
// is at or above the nearest one to a_j / sd and each element's error can only fall as k grows; once
// s_k >= sd (1 + 2^-21) every scaled value lies below a_j / sd, every code is at or below the nearest
// one and the error can only rise.  The block error of Eq. 8 is therefore smallest at the last
// multiplier of the first kind, at the first of the second kind, or at one in between (the band is
// 2^-20 wide against a grid step of a hundredth: almost always empty): two multipliers in the typical
// case, where the grid has 101.
//
// Equal errors.  Two multipliers with the same codes are one outcome (the quantization scale is
// never stored).  Different codes of an element cost the same only when a_j / sd is exactly a
// rounding midpoint; because the band keeps the scaled value of such an element strictly above the
// midpoint before it and strictly below after it, the element holds its upper code for every
// multiplier before the band and its lower code for every one after, whatever the tie rule of
// the rounding: all of its free code changes happen among the multipliers of [ka, kb].  Those are
// scored in grid order with Algorithm 1's strict comparison, and outside [ka, kb] the error changes
// strictly with every code change, so the first minimum of the whole grid has the codes of the
// first minimum found here.

// Binary32 bounds of the band around sd = alpha * dv (the exact product): lo <= sd (1 - 2^-21) and
// hi >= sd (1 + 2^-21), by directed roundings.
__device__ __forceinline__ void divisor_band(float alpha, float dv, float& lo, float& hi) {
  lo = __fmul_rd(__fmul_rd(alpha, dv), 1.0f - 0x1p-21f);
  hi = __fmul_ru(__fmul_ru(alpha, dv), 1.0f + 0x1p-21f);
}

// The range [ka, kb] of multipliers that can win for a code whose band is [lo, hi], for any start
// index k: walks to the last multiplier with s_k <= lo, then on to the first with s_k >= hi.
__device__ __forceinline__ void winning_range(const float* s_beta, int n_beta, float alpha, float center, float lo,
                                           float hi, int k, int& ka, int& kb) {
  k = max(0, min(n_beta - 1, k));
  while (k >= 0 && grid_divisor(alpha, center, s_beta[k]) > lo) --k;
  while (k + 1 < n_beta && grid_divisor(alpha, center, s_beta[k + 1]) <= lo) ++k;
  ka = max(k, 0);
  kb = k + 1;
  while (kb < n_beta && grid_divisor(alpha, center, s_beta[kb]) < hi) ++kb;
  kb = min(kb, n_beta - 1);
}

// A block's winner of Eq. 8: error minus sum W^2, its sums, codes (signs included) and E4M3 code.
struct Winner {
  double g, A, B;
  unsigned int c0, c1;
  int d;
};

// One candidate of the search scored on the exact integer sums: codes (signs included), afix, 4B and
// e = rho * 4B - afix, which orders candidates of one E4M3 code like their errors.
struct Scored {
  unsigned int c0, c1, afix, b4;
  double e;
};
__device__ __forceinline__ void score_candidate(const Block& blk, const Fixed& fx, float s, double rho, Scored& o) {
  round_block(blk, recip_fast(s), o.c0, o.c1);
  code_sums(fx, o.c0, o.c1, o.afix, o.b4);
  o.e = fma(rho, uint_to_double(o.b4), -uint_to_double(o.afix));
}

// One iteration t of Algorithm 1 for every block: Eq. 5 (from stage-t sums), Eq. 6,
// App. B.3 candidate sets, Eq. 8 search, winner stored, stage-(t+1) sums accumulated.
// Codes and scale bytes are written when `emit` is set (the state after this iteration may
// be the one returned); the per-block sums are kept when `keep` is set (another iteration
// may follow).  Modes 1 and 2 are the shapes with one quantization scale per E4M3 code and at most two
// codes, whose passes are bound by HBM rather than by the candidate loop.  Mode 4 is the candidate
// grid of App. B.3 searched through winning_range: per E4M3 code only the multipliers that can win
// are rounded and scored, which gives the winner of the whole grid.
template <int kMode, bool kDet>   // 0: candidate grid, every multiplier visited; 1: one candidate scale (beta = 1), at most two
                       // codes; 2: the same with the coupled scale; 3: one candidate scale, any number of codes;
                       // 4: candidate grid, only the multipliers that can win; 5: the same for grids so short that
                       // a block's bracket often reaches past their first or last multiplier
__global__ void __launch_bounds__(kThreads, (kMode == 1 || kMode == 3) ? 3 : 2)
iterate_kernel(const __grid_constant__ Batch bt, int t, int reverse, int emit, int keep, int prev_grid) {
  constexpr bool kSingle = kMode == 1 || kMode == 2 || kMode == 3;
  __shared__ RingWithState ring;
  __shared__ Slots<3, kDet> slots;
  __shared__ float s_beta[kSingle ? 1 : SOAR_MAX_BETA];
  __shared__ float s_alpha[kMaxBatch];
  __shared__ double s_latest[kDet ? kMaxBatch : 1][3];
  __shared__ unsigned int s_run;
  constexpr bool det = kDet;
  if (threadIdx.x == 0) s_run = 0;
  if (det) {
    // this CTA's slots of the stage it will fill start at zero; the stage the previous pass filled is added up
    for (int i = threadIdx.x; i < bt.n * 3; i += kThreads) bt.t[i / 3].det->stage[(t + 1) & 1][i % 3][blockIdx.x] = 0.0;
    gather_stage(bt, t, prev_grid, s_latest);
  }
  __syncthreads();
  if (threadIdx.x < bt.n) {   // per tensor: still running?  its alpha for this iteration
    float a;
    int run;
    iteration_head(bt.t[threadIdx.x], t, a, run, det ? s_latest[threadIdx.x] : nullptr);
    s_alpha[threadIdx.x] = a;
    if (run) atomicOr(&s_run, 1u << threadIdx.x);
  }
  const int n_dq = bt.t[0].n_dq, n_beta = bt.t[0].n_beta;
  if (!kSingle) {
    for (int k = threadIdx.x; k < n_beta; k += kThreads)
      s_beta[k] = static_cast<float>((100.0 + static_cast<double>((k - n_beta / 2) * bt.t[0].beta_step_pct)) / 100.0);
  }
  slots_clear(slots);
  __syncthreads();
  if (s_run == 0) return;   // every tensor of the batch has stopped
  ring_init(ring);
  if (is_producer_warp()) {
    if (threadIdx.x == kTile) ring_produce(ring, bt, reverse, s_run);
    return;
  }
  float alpha = 1.0f;
  double alpha_d = 1.0;
  // mode 4: multiplier index of a scale ratio, k = (ratio - 1) * 100 / step + n_beta / 2
  const float k_scale = 100.0f / static_cast<float>(max(bt.t[0].beta_step_pct, 1));
  const float k_off = static_cast<float>(n_beta / 2) - k_scale;   // k = (dv / center) * k_scale + k_off

  double acc[3] = {0.0, 0.0, 0.0};   // num, den, gsum of stage t+1
  unsigned int wide = 0, unused_zeros = 0;
  int cur = -1;
  Tensor p = {};   // the current tensor's pointers and size, kept in registers
  const int flags = bt.t[0].flags;
  for (unsigned int n = 0;; ++n) {
    uint4 v0, v1;
    uint2 st;
    int ti = -1;
    unsigned int tile = 0;
    const int rc = ring_consume(ring, bt, n, v0, v1, ti, tile, &st);
    if (rc != 0 || ti != cur) {
      if (cur >= 0) {
        Ws* ws = bt.t[cur].ws;
        DetParts* dp = bt.t[cur].det;
        const int sb = (t + 1) & 1;
        double* const dst[3] = {det ? &dp->stage[sb][0][blockIdx.x] : &ws->num[t + 1],
                                det ? &dp->stage[sb][1][blockIdx.x] : &ws->den[t + 1],
                                det ? &dp->stage[sb][2][blockIdx.x] : &ws->gsum[t + 1]};
        slots_add(slots, cur, acc, dst);
        add_counters(ws, unused_zeros, wide);
      }
      if (rc != 0) break;
      cur = ti;
      alpha = s_alpha[ti];
      alpha_d = static_cast<double>(alpha);
      if (kMode != 0) p = tensor_view(bt.t[ti]);
    }
    // the long candidate loop does better re-reading these from the parameter block per tile than
    // carrying them in registers
    if (kMode == 0) p = tensor_view(bt.t[ti]);
    const unsigned int b = tile * kTile + threadIdx.x;
    if (b >= p.nblk || (st.y >> 16) == 0) continue;   // past the end, or an all-zero block: nothing to optimise
    Block blk;
    unpack_block(v0, v1, blk);
    int d_lo, d_hi;
    const float center = block_center(st, alpha, n_dq, (flags & SOAR_FLAG_KEEP_BLOCK_SCALE) != 0, d_lo, d_hi);
    const int dc0 = clip_code(d_lo), dc1 = clip_code(d_lo + 1);
    const double sd0 = alpha_d * static_cast<double>(e4m3_value(dc0));
    const double sd1 = alpha_d * static_cast<double>(e4m3_value(dc1));
    Fixed fx;
    make_fixed(blk, fx);
    double best, bestA, bestB;
    int best_d = dc0;
    unsigned int best0, best1;
    if (kMode == 2) {
      // beta = 1 and the coupled scale of Sec. 3.2: each E4M3 candidate rounds the block with its
      // own value and is scored with it
      const float r0 = recip_scale(alpha, e4m3_value(dc0));
      round_block(blk, r0, best0, best1);
      block_sums(blk, fx, r0, best0, best1, bestA, bestB, wide);
      best = sd0 * fma(sd0, bestB, -2.0 * bestA);
      if (n_dq == 2) {
        const float r1 = recip_scale(alpha, e4m3_value(dc1));
        unsigned int c0, c1;
        double A, B;
        round_block(blk, r1, c0, c1);
        block_sums(blk, fx, r1, c0, c1, A, B, wide);
        const double g1 = sd1 * fma(sd1, B, -2.0 * A);
        if (g1 < best) { best = g1; best_d = dc1; bestA = A; bestB = B; best0 = c0; best1 = c1; }
      }
    } else if (kSingle) {
      // one quantization scale (beta = 1): the codes are fixed, only the E4M3 code is chosen
      const float r = recip_scale(alpha, center);
      round_block(blk, r, best0, best1);
      block_sums(blk, fx, r, best0, best1, bestA, bestB, wide);
      const double A2 = -2.0 * bestA;
      best = sd0 * fma(sd0, bestB, A2);               // block error minus sum W^2
      if (n_dq >= 2) {
        const double g1 = sd1 * fma(sd1, bestB, A2);
        if (g1 < best) { best = g1; best_d = dc1; }
      }
      if (kMode == 3) {
        for (int d = d_lo + 2; d <= d_hi; ++d) {      // wider code windows (App. B.3 with more than two codes)
          const int dc = clip_code(d);
          const double sd = alpha_d * static_cast<double>(e4m3_value(dc));
          const double g = sd * fma(sd, bestB, A2);
          if (g < best) { best = g; best_d = dc; }
        }
      }
    } else if (kMode == 4 || kMode == 5) {
      const int nd = d_hi - d_lo + 1;
      {
        // Typical block: two E4M3 codes at most, each with exactly two multipliers that can win (the one
        // just below value(code) / center and its successor), the exact integer sums valid and the
        // fast reciprocal in range for the whole grid.  Those four candidates are scored in straight
        // line; any other block takes the loops below.
        const bool second = nd == 2 && dc1 != dc0;
        const float per_center = __fdividef(k_scale, center);
        const float dv0 = e4m3_value(dc0), dv1 = e4m3_value(dc1);
        float lo0, hi0, lo1, hi1;
        divisor_band(alpha, dv0, lo0, hi0);
        divisor_band(alpha, dv1, lo1, hi1);
        const int k0 = max(0, min(n_beta - 2, __float2int_rd(__fmaf_rn(dv0, per_center, k_off))));
        const int k1 = max(0, min(n_beta - 2, __float2int_rd(__fmaf_rn(dv1, per_center, k_off))));
        const float s00 = grid_divisor(alpha, center, s_beta[k0]), s01 = grid_divisor(alpha, center, s_beta[k0 + 1]);
        const float s10 = grid_divisor(alpha, center, s_beta[k1]), s11 = grid_divisor(alpha, center, s_beta[k1 + 1]);
        // the four divisors lie between s00 and s11 (or s01 without a second code): those two bound the range
        // of the fast reciprocal, and the smallest one decides whether the exact integer sums hold
        const float s_hi = second ? s11 : s01;
        bool direct = nd <= 2 && fx.ok && recip_fast_ok(s00) && recip_fast_ok(s_hi) &&
                      __fmul_rn(blk.bmax, recip_fast(s00)) <= 32.0f;
        // Where the grid ends before the band does, one multiplier is all that can win: the first one when
        // even its divisor lies beyond the band, the last one when even its divisor lies before it.  The
        // pair then holds that multiplier twice.
        // (Mode 5 only: a grid that spans 0.85 .. 1.15 holds the whole bracket of every regular block.)
        const bool low0 = kMode == 5 && k0 == 0 && s00 >= hi0, high0 = kMode == 5 && k0 == n_beta - 2 && s01 <= lo0;
        const bool low1 = kMode == 5 && k1 == 0 && s10 >= hi1, high1 = kMode == 5 && k1 == n_beta - 2 && s11 <= lo1;
        direct = direct && ((s00 <= lo0 && s01 >= hi0) || low0 || high0);
        if (second) direct = direct && ((s10 <= lo1 && s11 >= hi1) || low1 || high1);
        if (direct) {
          // error minus sum W^2 = 2 sd unit (rho * 4B - afix) with rho = sd / (8 unit): per code the two
          // candidates are ranked on the exact integer sums, the codes' winners compared once
          Scored a, c;
          score_candidate(blk, fx, high0 ? s01 : s00, sd0 * fx.inv8, a);
          {
            Scored b2;
            score_candidate(blk, fx, low0 ? s00 : s01, sd0 * fx.inv8, b2);
            if (b2.e < a.e) a = b2;
          }
          double ga = 2.0 * sd0 * fx.unit * a.e;
          best_d = dc0;
          if (second) {
            score_candidate(blk, fx, high1 ? s11 : s10, sd1 * fx.inv8, c);
            Scored b2;
            score_candidate(blk, fx, low1 ? s10 : s11, sd1 * fx.inv8, b2);
            const bool later = b2.e < c.e;
            if (later) c = b2;
            const double gc = 2.0 * sd1 * fx.unit * c.e;
            // equal errors: the earlier multiplier, as in grid order (k1 >= k0 always)
            if (gc < ga) { ga = gc; a = c; best_d = dc1; }
          }
          best = ga;
          best0 = a.c0;
          best1 = a.c1;
          bestA = uint_to_double(a.afix) * fx.unit;
          bestB = uint_to_double(a.b4) * 0.25;
        } else {
          best = __longlong_as_double(0x7FF0000000000000ll);
          bestA = bestB = 0.0;
          best0 = best1 = 0u;
          int best_k = 0, prev = -1;
          for (int d = d_lo; d <= d_hi; ++d) {
            const int dc = clip_code(d);
            if (dc == prev) continue;   // clipping at the ends of the E4M3 range repeats a code
            prev = dc;
            const float dv = e4m3_value(dc);
            const double sd = alpha_d * static_cast<double>(dv);
            float lo, hi;
            divisor_band(alpha, dv, lo, hi);
            int ka, kb;
            winning_range(s_beta, n_beta, alpha, center, lo, hi, __float2int_rd(__fmaf_rn(dv, per_center, k_off)), ka,
                          kb);
            for (int k = ka; k <= kb; ++k) {
              const float sk = grid_divisor(alpha, center, s_beta[k]);
              const float r = recip_fast_ok(sk) ? recip_fast(sk) : __frcp_rn(sk);
              unsigned int c0, c1;
              double A, B;
              round_block(blk, r, c0, c1);
              block_sums(blk, fx, r, c0, c1, A, B, wide);
              const double g = sd * fma(sd, B, -2.0 * A);
              // equal errors: the earlier multiplier, then the smaller code, as in grid order
              if (g < best || (g == best && k < best_k)) {
                best = g; bestA = A; bestB = B; best0 = c0; best1 = c1; best_d = dc; best_k = k;
              }
            }
          }
        }
      }
    } else {
      // Eq. 8 over beta ascending, then scale code ascending; strict '<' keeps the first
      // minimum.  Every candidate is scored in full, with no test for "same codes as the
      // previous beta": under SIMT such a test only saves work when all 32 blocks of a warp
      // pass it at once, and it costs instructions on every candidate.  The loop keeps just
      // the best error and its (beta, code) index; the winner is re-made once at the end.
      best = __longlong_as_double(0x7FF0000000000000ll);
      int best_key = 0;
      const int nd = d_hi - d_lo + 1;
      // the reciprocal scale falls as beta grows, so the first candidate decides whether the
      // exact integer sums hold for all of them
      const bool coupled = (flags & SOAR_FLAG_COUPLED_SCALE) != 0;
      const bool all_narrow = fx.ok && __fmul_rn(blk.bmax, recip_scale(alpha, __fmul_rn(center, s_beta[0]))) <= 32.0f;
      // the products alpha * center * beta are monotone in beta: the end points bound them all
      const bool fast_rcp = recip_fast_ok(__fmul_rn(alpha, __fmul_rn(center, s_beta[0]))) &&
                            recip_fast_ok(__fmul_rn(alpha, __fmul_rn(center, s_beta[n_beta - 1])));
      if (all_narrow && nd <= 2 && !coupled && fast_rcp) {
        // error minus sum W^2 = sd^2 B - 2 sd A = q * (rho * (4B) - afix)  with  q = 2 sd unit > 0 and
        // rho = sd / (8 unit): per E4M3 code the candidates are ranked by rho * 4B - afix alone (one fma),
        // and the two codes' winners are compared once after the loop
        const double rho0 = sd0 * fx.inv8, rho1 = sd1 * fx.inv8;
        double h0 = best, h1 = best;
        int k0 = 0, k1 = 0;
        float mag[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) mag[j] = fabsf(blk.w[j]);
        for (int k = 0; k < n_beta; ++k) {
          const float r = recip_fast(__fmul_rn(alpha, __fmul_rn(center, s_beta[k])));
          unsigned int afix, b4;
          magnitude_sums(mag, fx, r, afix, b4);
          const double ad = uint_to_double(afix), bd = uint_to_double(b4);
          const double e0 = fma(rho0, bd, -ad);
          if (e0 < h0) { h0 = e0; k0 = k; }
          if (nd == 2) {
            const double e1 = fma(rho1, bd, -ad);
            if (e1 < h1) { h1 = e1; k1 = k; }
          }
        }
        const double g0 = 2.0 * sd0 * fx.unit * h0;
        const double g1 = (nd == 2) ? 2.0 * sd1 * fx.unit * h1 : best;
        // first minimum in (beta, code) order
        const bool second = g1 < g0 || (g1 == g0 && k1 < k0);
        best = second ? g1 : g0;
        best_key = second ? 2 * k1 + 1 : 2 * k0;
      } else {
        // general form: any number of E4M3 candidates, scales far below the block maximum, and the
        // coupled arm of Sec. 3.2, where each E4M3 candidate rounds the block with its own value
        for (int k = 0; k < n_beta; ++k) {
          float r = recip_scale(alpha, __fmul_rn(center, s_beta[k]));
          unsigned int c0, c1;
          double A = 0.0, B = 0.0;
          if (!coupled) {
            round_block(blk, r, c0, c1);
            block_sums(blk, fx, r, c0, c1, A, B, wide);
          }
          for (int d = 0; d < nd; ++d) {
            const float dv = e4m3_value(clip_code(d_lo + d));
            if (coupled) {
              r = recip_scale(alpha, __fmul_rn(dv, s_beta[k]));
              round_block(blk, r, c0, c1);
              block_sums(blk, fx, r, c0, c1, A, B, wide);
            }
            const double sd = alpha_d * static_cast<double>(dv);
            const double g = sd * fma(sd, B, -2.0 * A);
            if (g < best) { best = g; best_key = (nd <= 2 ? 2 : nd) * k + d; }
          }
        }
      }
      // the winner, made again from its index
      const int per = nd <= 2 ? 2 : nd;
      const int bk = best_key / per;
      best_d = clip_code(d_lo + (best_key - bk * per));
      const float r = recip_scale(alpha, __fmul_rn(coupled ? e4m3_value(best_d) : center, s_beta[bk]));
      round_block(blk, r, best0, best1);
      unsigned int unused = 0;
      block_sums(blk, fx, r, best0, best1, bestA, bestB, unused);
    }
    // The winner: codes and scale out, sums kept for the next iteration's Eq. 6.
    if (emit) {
      reinterpret_cast<uint2*>(p.packed)[b] = make_uint2(best0, best1);
      p.scales[b] = static_cast<uint8_t>(best_d);
    }
    if (keep)
      p.state[b] = make_uint2(__float_as_uint(static_cast<float>(bestA)),
                              static_cast<unsigned int>(bestB * 4.0) | (static_cast<unsigned int>(best_d) << 16));
    const double vd = static_cast<double>(e4m3_value(best_d));
    acc[0] = fma(bestA, vd, acc[0]);
    acc[1] = fma(bestB * vd, vd, acc[1]);
    acc[2] += best;
  }
}

// Where each tensor of a batch wants its alpha and its report (report may be null).
struct Reports {
  float* alpha[kMaxBatch];
  soar_result* result[kMaxBatch];
};

// Replays the early-stop rule over the stage sums, writes alpha and the report; one CTA per tensor.
__global__ void __launch_bounds__(128) finalize_kernel(const __grid_constant__ Batch bt,
                                                       const __grid_constant__ Reports rp, int prev_grid) {
  const Params& p = bt.t[blockIdx.x];
  float* out_alpha = rp.alpha[blockIdx.x];
  soar_result* res = rp.result[blockIdx.x];
  __shared__ double s_num[SOAR_MAX_ITERS + 1], s_den[SOAR_MAX_ITERS + 1], s_sse[SOAR_MAX_ITERS + 1];
  __shared__ double s_ta[SOAR_MAX_ITERS + 1];
  __shared__ int s_iters;
  if (p.det != nullptr) {
    // deterministic mode: the stage the last pass filled is still in the per-CTA slots; this CTA (the
    // only one working on this tensor) adds them up in order and files them in the header
    if (threadIdx.x < 32) {
      int filled = 1;
      if (p.max_iters > 0) {
        float unused;
        iteration_head(p, p.max_iters - 1, unused, filled);
      }
      if (filled) {
        double v[3];
#pragma unroll
        for (int i = 0; i < 3; ++i) v[i] = ordered_sum(p.det->stage[p.max_iters & 1][i], prev_grid);
        if (threadIdx.x == 0) {
          p.ws->num[p.max_iters] = v[0];
          p.ws->den[p.max_iters] = v[1];
          p.ws->gsum[p.max_iters] = v[2];
        }
      }
    }
    __threadfence_block();
    __syncthreads();
  }
  const Ws* ws = p.ws;
  const unsigned int amax_bits = ws->amax_bits;
  const int st = status_from_amax(amax_bits);
  for (int i = threadIdx.x; i <= SOAR_MAX_ITERS; i += blockDim.x) {
    const bool used = i <= p.max_iters;
    s_num[i] = used ? ws->num[i] : 0.0;
    s_den[i] = used ? ws->den[i] : 0.0;
    s_sse[i] = (used && st == 0) ? stage_sse(ws, i) : 0.0;
    s_ta[i] = 0.0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float alpha = (st & SOAR_STATUS_ZERO_TENSOR) ? 1.0f : __fdiv_rn(bits_to_mag(amax_bits), 2688.0f);
    int iters = 0;
    s_ta[0] = static_cast<double>(alpha);
    if (st == 0 && ws->error == 0) {
      double prev = s_sse[0];
      for (int i = 0; i < p.max_iters; ++i) {
        if (s_den[i] > 0.0 && !(p.flags & SOAR_FLAG_KEEP_ALPHA)) alpha = static_cast<float>(s_num[i] / s_den[i]);
        const double cur = s_sse[i + 1];
        iters = i + 1;
        s_ta[iters] = static_cast<double>(alpha);
        if (stops_after(prev, cur, p.early_stop_rel)) break;
        prev = cur;
      }
    }
    s_iters = iters;
    *out_alpha = alpha;
    if (res != nullptr) {
      res->status = st | ((ws->error & kErrWait) ? SOAR_STATUS_INTERNAL : 0) |
                    ((ws->error & kErrWeight) ? SOAR_STATUS_BAD_WEIGHT : 0);
      res->iters_run = iters;
      res->alpha = alpha;
      res->amax = bits_to_mag(amax_bits);
      res->sse = s_sse[iters];
      res->sse_init = s_sse[0];
      res->sumsq = (st & SOAR_STATUS_ZERO_TENSOR) ? 0.0 : ws->sumsq;
      res->zero_blocks = static_cast<int64_t>(ws->zero_blocks);
      res->wide_candidates = static_cast<int64_t>(ws->wide);
    }
  }
  __syncthreads();
  if (res != nullptr) {
    const int iters = s_iters;
    for (int i = threadIdx.x; i <= SOAR_MAX_ITERS; i += blockDim.x) {
      res->trace_alpha[i] = (i <= iters) ? s_ta[i] : 0.0;
      res->trace_sse[i] = (i <= iters) ? s_sse[i] : 0.0;
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

// Eq. 3-4 on stored outputs: sum (w - q s)^2 and sum w^2, one binary64 fma per term, with the
// bf16 values widened by the conversion instruction (which runs beside the integer and
// binary64 pipes) and the signed E2M1 values read from a 16-entry table in shared memory.
// A wait that gave up turns the results into NaN.  kWeighted multiplies every term by its
// column's weight h_j.
template <bool kWeighted>
__global__ void __launch_bounds__(kThreads) dequant_error_kernel(const __grid_constant__ Batch bt,
                                                                 const uint8_t* scales, int swizzled,
                                                                 unsigned int col_tiles, const float* alpha_ptr,
                                                                 const float* h, double* out_sse,
                                                                 double* out_sumsq) {
  __shared__ Ring ring;
  __shared__ Slots<2> slots;
  __shared__ double s_q[16];
  const Params& p = bt.t[0];
  slots_clear(slots);
  if (threadIdx.x < 16) {
    const double mag = static_cast<double>(e2m1_code_value(threadIdx.x & 7u));
    s_q[threadIdx.x] = (threadIdx.x & 8u) ? -mag : mag;
  }
  ring_init(ring);
  if (is_producer_warp()) {
    if (threadIdx.x == kTile) ring_produce(ring, bt, 0, 1u);
    return;
  }
  const double alpha_d = static_cast<double>(*alpha_ptr);
  double acc[2] = {0.0, 0.0};
  for (unsigned int n = 0;; ++n) {
    uint4 v0, v1;
    int ti;
    unsigned int tile;
    if (ring_consume(ring, bt, n, v0, v1, ti, tile) != 0) break;
    const unsigned int b = tile * kTile + threadIdx.x;
    if (b >= p.nblk) continue;
    const uint2 cw = reinterpret_cast<const uint2*>(p.packed)[b];
    int dc;
    if (swizzled) {
      const unsigned int row = b / p.nbc, cb = b - row * p.nbc;
      dc = scales[swizzled_offset(row, cb, col_tiles)];
    } else {
      dc = scales[b];
    }
    const double s = alpha_d * static_cast<double>(e4m3_value(dc & 0x7F));
    const unsigned int u[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
    double hd[16];
    if (kWeighted) load_weights(h, b % p.nbc, hd);
    double e0 = 0.0, e1 = 0.0, q0 = 0.0, q1 = 0.0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const double wl = static_cast<double>(__uint_as_float(u[i] << 16));
      const double wh = static_cast<double>(__uint_as_float(u[i] & 0xFFFF0000u));
      const unsigned int word = (i < 4) ? cw.x : cw.y;
      const double ql = s_q[(word >> (8 * (i & 3))) & 0xFu], qh = s_q[(word >> (8 * (i & 3) + 4)) & 0xFu];
      const double dl = fma(-ql, s, wl), dh = fma(-qh, s, wh);
      if (kWeighted) {
        e0 = fma(hd[2 * i], dl * dl, e0);
        e1 = fma(hd[2 * i + 1], dh * dh, e1);
        q0 = fma(hd[2 * i], wl * wl, q0);
        q1 = fma(hd[2 * i + 1], wh * wh, q1);
      } else {
        e0 = fma(dl, dl, e0);
        e1 = fma(dh, dh, e1);
        q0 = fma(wl, wl, q0);
        q1 = fma(wh, wh, q1);
      }
    }
    acc[0] += e0 + e1;
    acc[1] += q0 + q1;
  }
  const bool failed = *static_cast<volatile int*>(&ring.fail) != 0;
  if (failed) acc[0] = acc[1] = __longlong_as_double(0x7FF8000000000000ll);
  double* const dst[2] = {out_sse, out_sumsq};
  slots_add(slots, 0, acc, dst);
}

// ------------------------------------------------------------------ column-weighted objective
//
// Sec. 5 proposes to minimise the output distortion ||(W - What) X||^2 in CJSO and DSS; its
// diagonal form is sum_ij h_j (W_ij - What_ij)^2 with h_j the second moment of input channel j.
// Algorithm 1 is unchanged except that the block sums carry the weights,
//   A = sum h_j |w_j| m_j,   B = sum h_j m_j^2,
// in Eq. 5, Eq. 6 and the error of Eq. 8.  The weights are arbitrary binary32 numbers, so the
// integer dot products of the unweighted kernels do not apply: the sums are binary64, taken in
// element order (each product is exact: 24 + 8 + 2 and 24 + 4 significant bits), and the state
// kept between iterations is {A, B} in binary64 plus the scale code.

struct Weighted {
  const float* h;    // cols weights
  double2* sums;     // per block {A, B} of the current codes; null when T == 0
  uint8_t* code;     // per block stored scale code (0: all-zero block); null when T == 0
};
// One launch works on up to kMaxBatch matrices (see Batch): entry i belongs to bt.t[i].
struct WeightedBatch {
  Weighted t[kMaxBatch];
};

// A and B of a code vector (sign bits ignored) for hw[j] = h_j |w_j| and hd[j] = h_j.
__device__ __forceinline__ void weighted_sums(const double (&hw)[16], const double (&hd)[16], unsigned int c0,
                                              unsigned int c1, double& A, double& B) {
  const unsigned int m0 = c0 & 0x77777777u, m1 = c1 & 0x77777777u;
  const unsigned int t[4] = {twice_magnitude_x4(m0), twice_magnitude_x4(m0 >> 16), twice_magnitude_x4(m1),
                             twice_magnitude_x4(m1 >> 16)};
  double a = 0.0, b = 0.0;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const double dm = uint_to_double_bits((t[j >> 2] >> (8 * (j & 3))) & 0xFFu);   // 2 m_j
    a = fma(hw[j], dm, a);
    b = fma(hd[j], dm * dm, b);
  }
  // halving every term halves every partial sum exactly
  A = 0.5 * a;
  B = 0.25 * b;
}

// The same sums for ranking candidates: two interleaved partial chains per sum instead of one
// sixteen-long chain of dependent additions.  The result may differ from weighted_sums in the
// last bit, which only a tie between candidates could feel.
__device__ __forceinline__ void weighted_sums_split(const double (&hw)[16], const double (&hd)[16], unsigned int c0,
                                                    unsigned int c1, double& A, double& B) {
  const unsigned int t[4] = {twice_magnitude_x4(c0), twice_magnitude_x4(c0 >> 16), twice_magnitude_x4(c1),
                             twice_magnitude_x4(c1 >> 16)};
  double a[2] = {0.0, 0.0}, b[2] = {0.0, 0.0};
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const double dm = uint_to_double_bits((t[j >> 2] >> (8 * (j & 3))) & 0xFFu);
    a[j & 1] = fma(hw[j], dm, a[j & 1]);
    b[j & 1] = fma(hd[j], dm * dm, b[j & 1]);
  }
  A = 0.5 * (a[0] + a[1]);
  B = 0.25 * (b[0] + b[1]);
}

// A and B of a code vector (sign bits ignored) from the block's sixteen column weights and signed
// elements, in element order like weighted_sums and with the same roundings, but widening each
// weight and magnitude where it is used, so that only a few binary64 values are live at a time.
__device__ __forceinline__ void weighted_sums_streamed(const float (&h)[16], const float (&w)[16], unsigned int c0,
                                                       unsigned int c1, double& A, double& B) {
  const unsigned int m0 = c0 & 0x77777777u, m1 = c1 & 0x77777777u;
  const unsigned int t[4] = {twice_magnitude_x4(m0), twice_magnitude_x4(m0 >> 16), twice_magnitude_x4(m1),
                             twice_magnitude_x4(m1 >> 16)};
  double a = 0.0, b = 0.0;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const double dm = uint_to_double_bits((t[j >> 2] >> (8 * (j & 3))) & 0xFFu);   // 2 m_j
    const double hd = static_cast<double>(h[j]);
    a = fma(hd * static_cast<double>(fabsf(w[j])), dm, a);
    b = fma(hd, dm * dm, b);
  }
  A = 0.5 * a;
  B = 0.25 * b;
}

// hd[j] = h_j and hw[j] = h_j |w_j| of a block, binary64 (both exact).
__device__ __forceinline__ void block_weights(const float* h, unsigned int cb, const Block& mags, double (&hd)[16],
                                              double (&hw)[16]) {
  load_weights(h, cb, hd);
#pragma unroll
  for (int j = 0; j < 16; ++j) hw[j] = hd[j] * static_cast<double>(mags.w[j]);
}

__device__ __forceinline__ bool weight_ok(float h) {
  return h == 0.0f || (h >= 0x1p-20f && h <= 0x1p20f);
}

// Eq. 1's tensor maximum, sum h_j W^2 for the error report, and the check of the weights.
__global__ void __launch_bounds__(kThreads, 2)
weighted_amax_kernel(const __grid_constant__ Batch bt, const __grid_constant__ WeightedBatch wb) {
  __shared__ Ring ring;
  __shared__ Slots<1> slots;
  slots_clear(slots);
  ring_init(ring);
  if (is_producer_warp()) {
    if (threadIdx.x == kTile) ring_produce(ring, bt, 0, 0xFFFFFFFFu);
    return;
  }
  unsigned int mx = 0, nblk = 0, nbc = 1;
  const float* h = nullptr;
  bool bad = false;
  double sq[1] = {0.0};
  int cur = -1;
  for (unsigned int n = 0;; ++n) {
    uint4 v0, v1;
    int ti = -1;
    unsigned int tile = 0;
    const int rc = ring_consume(ring, bt, n, v0, v1, ti, tile);
    if (rc != 0 || ti != cur) {
      if (cur >= 0) {   // leaving tensor `cur`: hand over its maximum, its sum and the outcome of the weight check
        mx = __reduce_max_sync(0xFFFFFFFFu, mx);
        const bool any_bad = __any_sync(0xFFFFFFFFu, bad);
        if ((threadIdx.x & 31) == 0) {
          if (mx) atomicMax(&bt.t[cur].ws->amax_bits, mx);
          if (any_bad) atomicOr(&bt.t[cur].ws->error, kErrWeight);
        }
        double* const dst[1] = {&bt.t[cur].ws->sumsq};
        slots_add(slots, cur, sq, dst);
        mx = 0;
        bad = false;
      }
      if (rc != 0) break;
      cur = ti;
      nblk = bt.t[ti].nblk;
      nbc = bt.t[ti].nbc;
      h = wb.t[ti].h;
    }
    const unsigned int b = tile * kTile + threadIdx.x;
    if (b >= nblk) continue;
    const unsigned int u[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
    double hd[16];
    load_weights(h, b % nbc, hd);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      // magnitude bit patterns order like the magnitudes; NaN patterns lie above infinity's
      mx = max(mx, max(u[i] & 0x7FFFu, (u[i] >> 16) & 0x7FFFu));
      const double wl = static_cast<double>(__uint_as_float(u[i] << 16));
      const double wh = static_cast<double>(__uint_as_float(u[i] & 0xFFFF0000u));
      sq[0] = fma(hd[2 * i], wl * wl, sq[0]);
      sq[0] = fma(hd[2 * i + 1], wh * wh, sq[0]);
      bad = bad || !weight_ok(static_cast<float>(hd[2 * i])) || !weight_ok(static_cast<float>(hd[2 * i + 1]));
    }
  }
}

// Algorithm 1 "Initialization" (Eq. 1; the weights play no part in it), the first codes, and
// the weighted stage-0 sums of Eq. 5 and of the starting error.
__global__ void __launch_bounds__(kThreads, 2)
weighted_init_kernel(const __grid_constant__ Batch bt, const __grid_constant__ WeightedBatch wb, int reverse,
                     int final) {
  __shared__ Ring ring;
  __shared__ Slots<3> slots;
  slots_clear(slots);
  ring_init(ring);
  if (is_producer_warp()) {
    if (threadIdx.x == kTile) {
      unsigned int run = 0;
      for (int i = 0; i < bt.n; ++i)
        if (!(status_from_amax(bt.t[i].ws->amax_bits) & (SOAR_STATUS_NONFINITE | SOAR_STATUS_RANGE)) &&
            bt.t[i].ws->error == 0)
          run |= 1u << i;
      ring_produce(ring, bt, reverse, run);
    }
    return;
  }
  float alpha = 1.0f, six_alpha = 6.0f;
  double alpha_d = 1.0;
  double acc[3] = {0.0, 0.0, 0.0};   // num, den, gsum
  unsigned int zeros = 0, unused_wide = 0;
  int cur = -1;
  Tensor p = {};
  Weighted wq = {};
  unsigned int nbc = 1;
  for (unsigned int n = 0;; ++n) {
    uint4 v0, v1;
    int ti = -1;
    unsigned int tile = 0;
    const int rc = ring_consume(ring, bt, n, v0, v1, ti, tile);
    if (rc != 0 || ti != cur) {
      if (cur >= 0) {
        Ws* ws = bt.t[cur].ws;
        double* const dst[3] = {&ws->num[0], &ws->den[0], &ws->gsum[0]};
        slots_add(slots, cur, acc, dst);
        add_counters(ws, zeros, unused_wide);
      }
      if (rc != 0) break;
      cur = ti;
      const unsigned int amax_bits = bt.t[ti].ws->amax_bits;
      alpha = amax_bits == 0 ? 1.0f : __fdiv_rn(bits_to_mag(amax_bits), 2688.0f);
      six_alpha = __fmul_rn(alpha, 6.0f);
      alpha_d = static_cast<double>(alpha);
      p = tensor_view(bt.t[ti]);
      nbc = bt.t[ti].nbc;
      wq = wb.t[ti];
    }
    const unsigned int b = tile * kTile + threadIdx.x;
    if (b >= p.nblk) continue;
    Block blk;
    unpack_block(v0, v1, blk);
    uint2 codes;
    if (blk.bmax == 0.0f) {
      round_block(blk, 1.0f, codes.x, codes.y);
      reinterpret_cast<uint2*>(p.packed)[b] = codes;
      p.scales[b] = 0;
      if (wq.code != nullptr) wq.code[b] = 0;
      ++zeros;
      continue;
    }
    int c = e4m3_encode(__fdiv_rn(blk.bmax, six_alpha));
    c = max(c, 1);
    const float v = e4m3_value(c);
    round_block(blk, recip_scale(alpha, v), codes.x, codes.y);
    double hd[16], hw[16];
    load_weights(wq.h, b % nbc, hd);
#pragma unroll
    for (int j = 0; j < 16; ++j) hw[j] = hd[j] * static_cast<double>(fabsf(blk.w[j]));
    double A, B;
    weighted_sums(hw, hd, codes.x, codes.y, A, B);
    if (final) {
      reinterpret_cast<uint2*>(p.packed)[b] = codes;
      p.scales[b] = static_cast<uint8_t>(c);
    }
    if (wq.sums != nullptr) {
      wq.sums[b] = make_double2(A, B);
      wq.code[b] = static_cast<uint8_t>(c);
    }
    const double vd = static_cast<double>(v);
    const double sd = alpha_d * vd;
    acc[0] = fma(A, vd, acc[0]);
    acc[1] = fma(B * vd, vd, acc[1]);
    acc[2] += sd * fma(sd, B, -2.0 * A);
  }
}

// Eq. 8 for one block over the whole grid with binary64 sums for every candidate, first minimum in
// (beta, code) order; the winner is then made again with its signs and its sums in element order.
// Serves the coupled arm and the blocks whose candidates can cost exactly the same (see
// weighted_iterate_kernel).  Out of line and fed from memory (sixteen bf16 values at w16, the weights
// at h), so that nothing of it weighs on the registers of the common path.
__device__ __noinline__ void weighted_whole_grid_search(const float* h, unsigned int cb, const uint16_t* w16,
                                                        float alpha, float center, const float* s_beta, int n_beta,
                                                        int d_lo, int nd, bool coupled, bool fast_rcp, Winner* out) {
  Block blk, mags;
  {
    const uint4* src = reinterpret_cast<const uint4*>(w16);
    unpack_block(__ldg(src), __ldg(src + 1), blk);
#pragma unroll
    for (int j = 0; j < 16; ++j) mags.w[j] = fabsf(blk.w[j]);
  }
  const double alpha_d = static_cast<double>(alpha);
  double best = __longlong_as_double(0x7FF0000000000000ll);
  int best_key = 0;
  {
    double hd[16], hw[16];
    block_weights(h, cb, mags, hd, hw);
    for (int k = 0; k < n_beta; ++k) {
      unsigned int c0, c1;
      double A = 0.0, B = 0.0;
      if (!coupled) {
        const float s = __fmul_rn(alpha, __fmul_rn(center, s_beta[k]));
        round_block(mags, fast_rcp ? recip_fast(s) : __frcp_rn(s), c0, c1);
        weighted_sums_split(hw, hd, c0, c1, A, B);
      }
      for (int d = 0; d < nd; ++d) {
        const float dv = e4m3_value(clip_code(d_lo + d));
        if (coupled) {
          round_block(mags, recip_scale(alpha, __fmul_rn(dv, s_beta[k])), c0, c1);
          weighted_sums_split(hw, hd, c0, c1, A, B);
        }
        const double sd = alpha_d * static_cast<double>(dv);
        const double g = sd * fma(sd, B, -2.0 * A);
        if (g < best) { best = g; best_key = nd * k + d; }
      }
    }
  }
  Winner w;
  const int bk = best_key / nd;
  w.d = clip_code(d_lo + (best_key - bk * nd));
  round_block(blk, recip_scale(alpha, __fmul_rn(coupled ? e4m3_value(w.d) : center, s_beta[bk])), w.c0, w.c1);
  float hf[16];
  {
    const float4* src = reinterpret_cast<const float4*>(h) + static_cast<size_t>(cb) * 4;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float4 v = __ldg(src + q);
      hf[4 * q] = v.x; hf[4 * q + 1] = v.y; hf[4 * q + 2] = v.z; hf[4 * q + 3] = v.w;
    }
  }
  weighted_sums_streamed(hf, blk.w, w.c0, w.c1, w.A, w.B);
  w.g = best;
  *out = w;
}

// One iteration t of Algorithm 1 under the weighted objective: Eq. 5 from the stage-t sums,
// Eq. 6 per block from its stored {A, B}, App. B.3's candidates, Eq. 8 with the weighted
// error written as  sum h w^2 + sd^2 B - 2 sd A  (sd = alpha * candidate scale value), first
// minimum in (beta, code) order.  All of cfg's shapes and arms run through this one kernel, on up
// to kMaxBatch matrices per launch like the unweighted kernels.
__global__ void __launch_bounds__(kThreads, 2)
weighted_iterate_kernel(const __grid_constant__ Batch bt, const __grid_constant__ WeightedBatch wb, int t,
                        int reverse, int emit, int keep) {
  __shared__ Ring ring;
  __shared__ Slots<3> slots;
  __shared__ float s_beta[SOAR_MAX_BETA];
  __shared__ float s_alpha[kMaxBatch];
  __shared__ unsigned int s_run;
  if (threadIdx.x == 0) s_run = 0;
  __syncthreads();
  if (threadIdx.x < bt.n) {   // per tensor: still running?  its alpha for this iteration
    float a;
    int run;
    iteration_head(bt.t[threadIdx.x], t, a, run);
    s_alpha[threadIdx.x] = a;
    if (run) atomicOr(&s_run, 1u << threadIdx.x);
  }
  const Params& p0 = bt.t[0];
  const int n_dq = p0.n_dq, n_beta = p0.n_beta;
  for (int k = threadIdx.x; k < n_beta; k += kThreads)
    s_beta[k] = static_cast<float>((100.0 + static_cast<double>((k - n_beta / 2) * p0.beta_step_pct)) / 100.0);
  slots_clear(slots);
  __syncthreads();
  if (s_run == 0) return;   // every tensor of the batch has stopped (Sec. 4.1), or was rejected
  ring_init(ring);
  if (is_producer_warp()) {
    if (threadIdx.x == kTile) ring_produce(ring, bt, reverse, s_run);
    return;
  }
  float alpha = 1.0f;
  double alpha_d = 1.0;
  const bool coupled = (p0.flags & SOAR_FLAG_COUPLED_SCALE) != 0;
  const bool keep_scale = (p0.flags & SOAR_FLAG_KEEP_BLOCK_SCALE) != 0;
  // multiplier index of a scale ratio: k = (ratio - 1) * 100 / step + n_beta / 2
  const bool bracketed = p0.beta_step_pct >= 1 && n_beta >= 2;
  const float k_scale = 100.0f / static_cast<float>(max(p0.beta_step_pct, 1));
  const float k_off = static_cast<float>(n_beta / 2) - k_scale;
  double acc[3] = {0.0, 0.0, 0.0};   // num, den, gsum of stage t+1
  unsigned int exact_blocks = 0, unused_zeros = 0;
  int cur = -1;
  for (unsigned int n = 0;; ++n) {
    uint4 v0, v1;
    int ti = -1;
    unsigned int tile = 0;
    const int rc = ring_consume(ring, bt, n, v0, v1, ti, tile);
    if (rc != 0 || ti != cur) {
      if (cur >= 0) {
        Ws* ws = bt.t[cur].ws;
        double* const dst[3] = {&ws->num[t + 1], &ws->den[t + 1], &ws->gsum[t + 1]};
        slots_add(slots, cur, acc, dst);
        add_counters(ws, unused_zeros, exact_blocks);   // reported as soar_result.wide_candidates
      }
      if (rc != 0) break;
      cur = ti;
      alpha = s_alpha[ti];
      alpha_d = static_cast<double>(alpha);
    }
    // pointers and sizes of the current tensor are re-read from the parameter block per tile rather than
    // carried in registers across the scoring of the block
    const Params& p = bt.t[ti];
    const Weighted& wq = wb.t[ti];
    const unsigned int b = tile * kTile + threadIdx.x;
    if (b >= p.nblk) continue;
    const int d_cur = wq.code[b];
    if (d_cur == 0) continue;   // all-zero block
    const double2 ab = wq.sums[b];
    Block blk;
    unpack_block(v0, v1, blk);
    const unsigned int row = b / p.nbc, cb = b - row * p.nbc;
    // Eq. 6 (binary32 steps); a block whose weighted codes are all zero keeps its stored scale
    const float center = (ab.y > 0.0 && !keep_scale)
                             ? __fdiv_rn(static_cast<float>(ab.x), __fmul_rn(alpha, static_cast<float>(ab.y)))
                             : e4m3_value(d_cur);
    int d_lo, d_hi;
    candidate_window(center, n_dq, d_lo, d_hi);
    const int nd = d_hi - d_lo + 1;
    // the products alpha * center * beta are monotone in beta: the end points bound them all
    const bool fast_rcp = !coupled && recip_fast_ok(__fmul_rn(alpha, __fmul_rn(center, s_beta[0]))) &&
                          recip_fast_ok(__fmul_rn(alpha, __fmul_rn(center, s_beta[n_beta - 1])));
    float hf[16];
    {
      const float4* src = reinterpret_cast<const float4*>(wq.h) + static_cast<size_t>(cb) * 4;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float4 v = __ldg(src + q);
        hf[4 * q] = v.x; hf[4 * q + 1] = v.y; hf[4 * q + 2] = v.z; hf[4 * q + 3] = v.w;
      }
    }
    // The weighted error of element j, h_j (a_j - m sd)^2, is convex in m like the unweighted one, so per
    // E4M3 code only the multipliers of winning_range can win (see there).  When a column's weight is zero,
    // its code costs nothing whatever it is, and equal errors of different codes occur all along the grid:
    // such blocks, and the coupled arm, walk the whole grid.
    bool zero_weight = false;
#pragma unroll
    for (int j = 0; j < 16; ++j) zero_weight = zero_weight || hf[j] == 0.0f;
    unsigned int best0 = 0, best1 = 0;
    double bestA = 0.0, bestB = 0.0;
    int best_d = clip_code(d_lo);
    if (!coupled && bracketed && !zero_weight) {
      double best = __longlong_as_double(0x7FF0000000000000ll);
      int best_k = 0, prev = -1;
      const float per_center = __fdividef(k_scale, center);
      for (int d = d_lo; d <= d_hi; ++d) {
        const int dc = clip_code(d);
        if (dc == prev) continue;   // clipping at the ends of the E4M3 range repeats a code
        prev = dc;
        const float dv = e4m3_value(dc);
        const double sd = alpha_d * static_cast<double>(dv);
        float lo, hi;
        divisor_band(alpha, dv, lo, hi);
        int ka = max(0, min(n_beta - 2, __float2int_rd(__fmaf_rn(dv, per_center, k_off))));
        int kb = ka + 1;
        if (!(grid_divisor(alpha, center, s_beta[ka]) <= lo && grid_divisor(alpha, center, s_beta[kb]) >= hi))
          winning_range(s_beta, n_beta, alpha, center, lo, hi, ka, ka, kb);
        for (int k = ka; k <= kb; ++k) {
          const float sk = grid_divisor(alpha, center, s_beta[k]);
          unsigned int c0, c1;
          round_block(blk, fast_rcp ? recip_fast(sk) : __frcp_rn(sk), c0, c1);
          double A, B;
          weighted_sums_streamed(hf, blk.w, c0, c1, A, B);
          const double g = sd * fma(sd, B, -2.0 * A);
          // equal errors: the earlier multiplier, then the smaller code, as in grid order
          if (g < best || (g == best && k < best_k)) {
            best = g; bestA = A; bestB = B; best0 = c0; best1 = c1; best_d = dc; best_k = k;
          }
        }
      }
    } else {
      Winner w;
      weighted_whole_grid_search(wq.h, cb, p.W + static_cast<long long>(row) * p.ld + static_cast<long long>(cb) * 16,
                                 alpha, center, s_beta, n_beta, d_lo, nd, coupled, fast_rcp, &w);
      ++exact_blocks;
      best0 = w.c0;
      best1 = w.c1;
      bestA = w.A;
      bestB = w.B;
      best_d = w.d;
    }
    if (emit) {
      reinterpret_cast<uint2*>(p.packed)[b] = make_uint2(best0, best1);
      p.scales[b] = static_cast<uint8_t>(best_d);
    }
    if (keep) {
      wq.sums[b] = make_double2(bestA, bestB);
      wq.code[b] = static_cast<uint8_t>(best_d);
    }
    const double vd = static_cast<double>(e4m3_value(best_d));
    const double sd = alpha_d * vd;
    acc[0] = fma(bestA, vd, acc[0]);
    acc[1] = fma(bestB * vd, vd, acc[1]);
    acc[2] += sd * fma(sd, bestB, -2.0 * bestA);
  }
}

// ------------------------------------------------------------------ MXFP4 (Sec. 4.3, "DSS on MXFP4")
//
// The other microscaling format: E2M1 elements in blocks of 32 with one shared power-of-two
// scale (an E8M0 byte, value 2^(code - 127)) and no tensor-wide scale.  The paper reports results
// and no procedure; the reading built here (the oracle's) is Sec. 3.3 (i)-(ii) with alpha = 1:
//   plain rule  shared exponent floor(log2 bmax) - 2, elements rounded to nearest even, saturated;
//   search      high-precision scale D* = fl(bmax / 6) (Eq. 1); dequantization candidates the n_dq E8M0
//               values around D* (App. B.3's rule on powers of two; for two candidates the plain
//               exponent is always one of them); quantization candidates D* * beta_k on App. B.3's
//               grid; Eq. 8 over all pairs, first minimum in (beta, code) order.
// Two neighbouring threads share a block of 32, sixteen elements each, and exchange their maxima and
// block sums by shuffles inside the pair; everything else is the machinery of the NVFP4 kernels.
// Candidates with exactly equal errors are the rule here (a power-of-two scale and bf16 inputs put an
// element exactly on a rounding midpoint in a fifth of all blocks), so the search keeps the grid's
// order where it matters: see the comment in the kernel.  One pass over W, no workspace.

__device__ __forceinline__ double pair_sum(unsigned int pair_mask, double v) {
  return v + __shfl_xor_sync(pair_mask, v, 1);
}

template <bool kSearch>
__global__ void __launch_bounds__(kThreads, 2)
mx_kernel(const __grid_constant__ Batch bt, uint8_t* scales, soar_mx_result* res, double* gsum, int n_dq, int n_beta,
          int step_pct) {
  __shared__ Ring ring;
  __shared__ Slots<2> slots;
  __shared__ float s_beta[kSearch ? SOAR_MAX_BETA : 1];
  const Params& p = bt.t[0];
  if (kSearch)
    for (int k = threadIdx.x; k < n_beta; k += kThreads)
      s_beta[k] = static_cast<float>((100.0 + static_cast<double>((k - n_beta / 2) * step_pct)) / 100.0);
  slots_clear(slots);
  ring_init(ring);
  if (is_producer_warp()) {
    if (threadIdx.x == kTile) ring_produce(ring, bt, 0, 1u);
    return;
  }
  const unsigned int pair_mask = 3u << (threadIdx.x & 30u);
  const bool first_of_pair = (threadIdx.x & 1u) == 0u;
  // multiplier index of a scale ratio: k = (ratio - 1) * 100 / step + n_beta / 2
  const bool bracketed = kSearch && n_beta >= kBracketMinBeta && step_pct >= 1;
  const float k_scale = 100.0f / static_cast<float>(max(step_pct, 1));
  const float k_off = static_cast<float>(n_beta / 2) - k_scale;
  double acc[2] = {0.0, 0.0};   // error minus sum W^2; sum W^2
  unsigned int zeros = 0, wide = 0, mx = 0;
  for (unsigned int n = 0;; ++n) {
    uint4 v0, v1;
    int ti;
    unsigned int tile;
    if (ring_consume(ring, bt, n, v0, v1, ti, tile) != 0) break;
    const unsigned int b = tile * kTile + threadIdx.x;   // index of this thread's sixteen elements
    if (b >= p.nblk) continue;                           // pairs leave together: nblk is even
    const unsigned int u[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) mx = max(mx, max(u[i] & 0x7FFFu, (u[i] >> 16) & 0x7FFFu));
    {
      double s0 = 0.0, s1 = 0.0;
      sumsq_block(u, s0, s1);
      acc[1] += s0 + s1;
    }
    Block blk;
    unpack_block(v0, v1, blk);
    const float bmax = fmaxf(blk.bmax, __shfl_xor_sync(pair_mask, blk.bmax, 1));
    uint2 codes;
    int code = 0;
    if (!(bmax >= 0x1p-120f)) {
      // zero (or vanishing) block: scale code 0, zero codes with the inputs' sign bits
      round_block(blk, 0.0f, codes.x, codes.y);
      if (first_of_pair) ++zeros;
    } else {
      Fixed fx;
      make_fixed(blk, fx);
      double best;
      float best_r;
      if (!kSearch) {
        const int X = static_cast<int>(__float_as_uint(bmax) >> 23) - 129;   // floor(log2 bmax) - 2
        code = X + 127;
        best_r = __uint_as_float(static_cast<unsigned int>(127 - X) << 23);   // 2^-X
        unsigned int c0, c1;
        double A, B;
        round_block(blk, best_r, c0, c1);
        block_sums(blk, fx, best_r, c0, c1, A, B, wide);
        A = pair_sum(pair_mask, A);
        B = pair_sum(pair_mask, B);
        const double sd = __hiloint2double((code + 896) << 20, 0);   // 2^(code - 127)
        best = sd * fma(sd, B, -2.0 * A);
      } else {
        const float center = __fdiv_rn(bmax, 6.0f);
        const int cf = static_cast<int>(__float_as_uint(center) >> 23);      // biased: value 2^(cf - 127) <= center
        int d_lo, d_hi;
        if (n_dq <= 1) {
          const float mid = __uint_as_float((static_cast<unsigned int>(cf) << 23) | 0x400000u);   // 1.5 * 2^(cf - 127)
          d_lo = d_hi = center > mid ? cf + 1 : cf;
        } else {
          d_lo = cf - (n_dq / 2 - 1);
          d_hi = cf + n_dq / 2;
        }
        best = __longlong_as_double(0x7FF0000000000000ll);
        best_r = 1.0f;
        if (!bracketed) {
          // every multiplier in turn (grids of a few multipliers)
          for (int k = 0; k < n_beta; ++k) {
            const float r = recip_scale(1.0f, __fmul_rn(center, s_beta[k]));
            unsigned int c0, c1;
            double A, B;
            round_block(blk, r, c0, c1);
            block_sums(blk, fx, r, c0, c1, A, B, wide);
            A = pair_sum(pair_mask, A);
            B = pair_sum(pair_mask, B);
            int prev = -1;
            for (int d = d_lo; d <= d_hi; ++d) {
              const int dc = max(0, min(254, d));
              if (dc == prev) continue;   // clipping at the ends of the E8M0 range repeats a code
              prev = dc;
              const double sd = __hiloint2double((dc + 896) << 20, 0);
              const double g = sd * fma(sd, B, -2.0 * A);
              if (g < best) { best = g; best_r = r; code = dc; }
            }
          }
        } else {
          // Per E8M0 code only the multipliers around divisor = 2^(code - 127) can win (see winning_range's
          // comment above iterate_kernel).  With a power-of-two scale and bf16 inputs, elements sit exactly on
          // rounding midpoints in a fifth of all blocks, so equal errors of different codes are the rule here.
          // The band is therefore 2^-21 wide on each side: before it the scaled value of such an element lies
          // strictly above its midpoint for every multiplier (it keeps the upper code, whatever the tie rule),
          // after it strictly below, so all of those free code changes happen inside [ka, kb], where the
          // candidates are scored in grid order with the strict comparison of Algorithm 1; outside it the
          // error changes strictly whenever a code changes.  The first minimum in (multiplier, code) order
          // then has the codes of the first minimum found here.
          int best_k = 0, prev = -1;
          const float per_center = __fdividef(k_scale, center);
          for (int d = d_lo; d <= d_hi; ++d) {
            const int dc = max(0, min(254, d));
            if (dc == prev) continue;
            prev = dc;
            const double sd = __hiloint2double((dc + 896) << 20, 0);
            const float sdf = static_cast<float>(sd);                       // exact (2^-127 is a binary32 subnormal)
            const float lo = __fmul_rn(sdf, 1.0f - 0x1p-21f), hi = __fmul_rn(sdf, 1.0f + 0x1p-21f);
            int ka, kb;
            winning_range(s_beta, n_beta, 1.0f, center, lo, hi, __float2int_rd(__fmaf_rn(sdf, per_center, k_off)), ka, kb);
            for (int k = ka; k <= kb; ++k) {
              const float r = recip_scale(1.0f, __fmul_rn(center, s_beta[k]));
              unsigned int c0, c1;
              double A, B;
              round_block(blk, r, c0, c1);
              block_sums(blk, fx, r, c0, c1, A, B, wide);
              A = pair_sum(pair_mask, A);
              B = pair_sum(pair_mask, B);
              const double g = sd * fma(sd, B, -2.0 * A);
              // equal errors: the earlier multiplier, then the smaller code, as in grid order
              if (g < best || (g == best && k < best_k)) { best = g; best_r = r; code = dc; best_k = k; }
            }
          }
        }
      }
      round_block(blk, best_r, codes.x, codes.y);
      if (first_of_pair) acc[0] += best;
    }
    reinterpret_cast<uint2*>(p.packed)[b] = codes;
    if (first_of_pair) scales[b >> 1] = static_cast<uint8_t>(code);
  }
  mx = __reduce_max_sync(0xFFFFFFFFu, mx);
  if ((threadIdx.x & 31) == 0 && mx) atomicMax(&res->amax_bits, mx);
  unsigned int unused = 0;
  zeros = __reduce_add_sync(0xFFFFFFFFu, zeros);
  wide = __reduce_add_sync(0xFFFFFFFFu, wide);
  if ((threadIdx.x & 31) == 0) {
    if (zeros) atomicAdd(reinterpret_cast<unsigned long long*>(&res->zero_blocks), static_cast<unsigned long long>(zeros));
    if (wide) atomicAdd(reinterpret_cast<unsigned long long*>(&res->wide_candidates), static_cast<unsigned long long>(wide));
    if (*static_cast<volatile int*>(&ring.fail)) atomicOr(&res->status, SOAR_STATUS_INTERNAL);
  }
  (void)unused;
  double* const dst[2] = {gsum, &res->sumsq};
  slots_add(slots, 0, acc, dst);
}

// Status and error of an MXFP4 call from its sums.
__global__ void mx_finalize_kernel(soar_mx_result* res, const double* gsum) {
  const unsigned int amax_bits = res->amax_bits;
  int st = res->status;
  if (amax_bits >= 0x7F80u) st |= SOAR_STATUS_NONFINITE;
  if (amax_bits == 0) st |= SOAR_STATUS_ZERO_TENSOR;
  res->status = st;
  res->amax = bits_to_mag(amax_bits);
  res->sse = fmax(res->sumsq + *gsum, 0.0);
}

// Counts the binary32 inputs with biased exponent lo_exp..hi_exp (all 2^23 significands each)
// on which recip_fast differs from rcp.rn.
__global__ void selftest_reciprocal_kernel(unsigned int lo_exp, unsigned int hi_exp, unsigned long long* mismatches) {
  const unsigned long long total = static_cast<unsigned long long>(hi_exp - lo_exp + 1) << 23;
  unsigned long long bad = 0;
  for (unsigned long long i = blockIdx.x * static_cast<unsigned long long>(blockDim.x) + threadIdx.x; i < total;
       i += static_cast<unsigned long long>(gridDim.x) * blockDim.x) {
    const float s = __uint_as_float((lo_exp << 23) + static_cast<unsigned int>(i));
    if (__float_as_uint(recip_fast(s)) != __float_as_uint(__frcp_rn(s))) ++bad;
  }
  if (bad) atomicAdd(mismatches, bad);
}

// ------------------------------------------------------------------ host side

// Optional launch tracing for benchmarks: while enabled, every kernel this library launches
// is bracketed by two CUDA events on the launching stream.
enum KernelId {
  K_AMAX = 0, K_INIT, K_ITERATE, K_FINALIZE, K_SWIZZLE, K_DEQUANT_ERROR,
  K_WEIGHTED_AMAX, K_WEIGHTED_INIT, K_WEIGHTED_ITERATE, K_MX, K_COUNT
};
const char* const kKernelNames[K_COUNT] = {"amax_kernel",          "init_kernel",          "iterate_kernel",
                                           "finalize_kernel",      "swizzle_kernel",       "dequant_error_kernel",
                                           "weighted_amax_kernel", "weighted_init_kernel", "weighted_iterate_kernel",
                                           "mx_kernel"};
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

// Test hook (soar_debug_fail_waits): what the launches put into Batch::idle_producer.
int g_idle_producer = 0;

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

// Grid of a persistent kernel: every SM filled to the kernel's occupancy, never more CTAs
// than tiles.
template <typename K>
unsigned int persistent_grid(K kernel, unsigned int tiles, int threads) {
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, 0) != cudaSuccess || per_sm <= 0)
    per_sm = 2;
  unsigned int cap = static_cast<unsigned int>(sm_count() * per_sm);
  if (cap > static_cast<unsigned int>(kMaxGrid)) cap = kMaxGrid;   // the deterministic mode keeps one slot per CTA
  return tiles < cap ? (tiles ? tiles : 1u) : cap;
}

size_t round256(size_t n) { return (n + 255) / 256 * 256; }

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
  if ((cfg->flags & ~(SOAR_FLAG_COUPLED_SCALE | SOAR_FLAG_KEEP_ALPHA | SOAR_FLAG_KEEP_BLOCK_SCALE |
                      SOAR_FLAG_DETERMINISTIC)) != 0)
    return SOAR_ERR_INVALID_ARG;
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
    case SOAR_PRESET_CJSO_ONLY:
      cfg->max_iters = 15; cfg->early_stop_rel = 1e-3f; cfg->n_dq = 1; cfg->n_beta = 1;
      cfg->flags = SOAR_FLAG_COUPLED_SCALE;
      return SOAR_OK;
    case SOAR_PRESET_COUPLED_PAIR:
      cfg->max_iters = 15; cfg->early_stop_rel = 1e-3f; cfg->n_dq = 2; cfg->n_beta = 1;
      cfg->flags = SOAR_FLAG_COUPLED_SCALE;
      return SOAR_OK;
    case SOAR_PRESET_DSS_ONLY:
      cfg->max_iters = 1; cfg->early_stop_rel = 0.0f; cfg->n_dq = 2; cfg->n_beta = 101;
      cfg->flags = SOAR_FLAG_KEEP_ALPHA | SOAR_FLAG_KEEP_BLOCK_SCALE;
      return SOAR_OK;
    default:
      return SOAR_ERR_INVALID_ARG;
  }
}

size_t soar_workspace_bytes(int64_t rows, int64_t cols, const soar_cfg* cfg) {
  if (check_cfg(cfg) != SOAR_OK || rows <= 0 || cols <= 0 || cols % 16 != 0) return 0;
  const size_t nblk = static_cast<size_t>(rows) * static_cast<size_t>(cols / 16);
  size_t n = kWsFixedBytes;
  if (cfg->max_iters > 0) n += round256(nblk * sizeof(uint2));
  if (!(cfg->scale_layout & SOAR_SCALES_LINEAR)) n += round256(nblk);
  if (cfg->flags & SOAR_FLAG_DETERMINISTIC) n += round256(sizeof(DetParts));
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

size_t soar_batch_workspace_bytes(const soar_tensor_desc* tensors, int n, const soar_cfg* cfg) {
  if (tensors == nullptr || n <= 0) return 0;
  size_t total = 0;
  for (int i = 0; i < n; ++i) {
    const size_t b = soar_workspace_bytes(tensors[i].rows, tensors[i].cols, cfg);
    if (b == 0) return 0;
    total += b;
  }
  return total;
}

}  // extern "C"

namespace {

// Which launches a call makes: all of them (soar_quantize_batch), or one stage
// (soar_quantize_stage; iterations t_lo <= t < t_hi for kStageIterate).
enum : int { kStageAmax = 1, kStageInit = 2, kStageIterate = 4, kStageFinalize = 8, kStageAll = 15 };

int run_batch(const soar_tensor_desc* tensors, int n, const soar_cfg* cfg, void* workspace, size_t workspace_bytes,
              void* stream, int stages, int t_lo, int t_hi) {
  int rc = check_cfg(cfg);
  if (rc != SOAR_OK) return rc;
  if (tensors == nullptr || n <= 0) return SOAR_ERR_INVALID_ARG;
  const bool want_lin = (cfg->scale_layout & SOAR_SCALES_LINEAR) != 0;
  const bool want_sw = (cfg->scale_layout & SOAR_SCALES_SWIZZLED) != 0;
  const bool det = (cfg->flags & SOAR_FLAG_DETERMINISTIC) != 0;
  // a stage run alone leaves its sums in the per-CTA slots, which the caller of the stages cannot combine
  if (det && stages != kStageAll) return SOAR_ERR_UNSUPPORTED;
  for (int i = 0; i < n; ++i) {   // every argument is checked before anything is enqueued
    const soar_tensor_desc& d = tensors[i];
    rc = check_shape(d.W_bf16, d.rows, d.cols, d.ld);
    if (rc != SOAR_OK) return rc;
    if (d.out_fp4_packed == nullptr || d.out_global_fp32 == nullptr) return SOAR_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d.out_fp4_packed) % 16 != 0) return SOAR_ERR_UNSUPPORTED;
    if (want_lin && d.out_e4m3_scales == nullptr) return SOAR_ERR_INVALID_ARG;
    if (want_sw && d.out_e4m3_scales_sw == nullptr) return SOAR_ERR_INVALID_ARG;
  }
  const size_t need = soar_batch_workspace_bytes(tensors, n, cfg);
  if (workspace == nullptr || need == 0 || workspace_bytes < need) return SOAR_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return SOAR_ERR_UNSUPPORTED;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // workspace: the n headers first (one memset clears them all), then each tensor's arrays
  uint8_t* const headers = static_cast<uint8_t*>(workspace);
  uint8_t* next = headers + static_cast<size_t>(n) * kWsFixedBytes;
  if ((stages & kStageAmax) &&
      cudaMemsetAsync(headers, 0, static_cast<size_t>(n) * kWsFixedBytes, st) != cudaSuccess)
    return SOAR_ERR_CUDA;

  // one quantization scale per block: the codes are made once (any number of E4M3 codes scored on them;
  // the coupled arm, where every code rounds the block anew, only with at most two)
  const bool single = cfg->n_beta == 1 && (cfg->n_dq <= 2 || !(cfg->flags & SOAR_FLAG_COUPLED_SCALE));
  const bool may_stop = cfg->early_stop_rel > 0.0f;
  for (int first = 0; first < n; first += kMaxBatch) {
    Batch bt;
    Reports rp;
    memset(&bt, 0, sizeof(bt));
    memset(&rp, 0, sizeof(rp));
    bt.n = (n - first < kMaxBatch) ? n - first : kMaxBatch;
    bt.idle_producer = g_idle_producer;
    unsigned int tiles = 0;
    for (int j = 0; j < bt.n; ++j) {
      const soar_tensor_desc& d = tensors[first + j];
      Params& p = bt.t[j];
      p.W = static_cast<const uint16_t*>(d.W_bf16);
      p.packed = static_cast<uint8_t*>(d.out_fp4_packed);
      p.ws = reinterpret_cast<Ws*>(headers + static_cast<size_t>(first + j) * kWsFixedBytes);
      p.ld = d.ld;
      p.nbc = static_cast<unsigned int>(d.cols / 16);
      p.nblk = static_cast<unsigned int>(d.rows * (d.cols / 16));
      p.ntiles = (p.nblk + kTile - 1) / kTile;
      p.contiguous = (d.ld == d.cols) ? 1 : 0;
      p.state = nullptr;
      if (cfg->max_iters > 0) {
        p.state = reinterpret_cast<uint2*>(next);
        next += round256(static_cast<size_t>(p.nblk) * sizeof(uint2));
      }
      if (want_lin) {
        p.scales = static_cast<uint8_t*>(d.out_e4m3_scales);
      } else {
        p.scales = next;
        next += round256(p.nblk);
      }
      p.det = nullptr;
      if (det) {
        p.det = reinterpret_cast<DetParts*>(next);
        next += round256(sizeof(DetParts));
      }
      p.max_iters = cfg->max_iters;
      p.early_stop_rel = cfg->early_stop_rel;
      p.n_dq = cfg->n_dq;
      p.n_beta = cfg->n_beta;
      p.beta_step_pct = cfg->beta_step_pct;
      p.flags = cfg->flags;
      tiles += p.ntiles;
      bt.tile_end[j] = tiles;
      rp.alpha[j] = d.out_global_fp32;
      rp.result[j] = d.out_result;
    }
    for (int j = bt.n; j < kMaxBatch; ++j) bt.tile_end[j] = 0xFFFFFFFFu;   // never reached by a tile index
    bt.total_tiles = tiles;

    // Passes alternate direction over the tiles (amax forward, init backward, iteration t forward
    // for even t): each starts where the previous one ended, on data still in L2.
    const unsigned int g_amax = det ? persistent_grid(amax_kernel<true>, tiles, kThreads)
                                    : persistent_grid(amax_kernel<false>, tiles, kThreads);
    const unsigned int g_init = det ? persistent_grid(init_kernel<true>, tiles, kThreads)
                                    : persistent_grid(init_kernel<false>, tiles, kThreads);
    unsigned int g_last = g_init;   // grid of the pass whose sums the next kernel's head reads
    if (stages & kStageAmax) {
      ScopedLaunch sl(K_AMAX, st);
      if (det) amax_kernel<true><<<g_amax, kThreads, 0, st>>>(bt, 0);
      else amax_kernel<false><<<g_amax, kThreads, 0, st>>>(bt, 0);
    }
    if (stages & kStageInit) {
      ScopedLaunch sl(K_INIT, st);
      const int final = cfg->max_iters == 0 ? 1 : 0;
      if (det) init_kernel<true><<<g_init, kThreads, 0, st>>>(bt, 1, final, static_cast<int>(g_amax));
      else init_kernel<false><<<g_init, kThreads, 0, st>>>(bt, 1, final, static_cast<int>(g_amax));
    }
    if (stages & kStageIterate) {
      // a grid of several multipliers with one quantization scale per multiplier: only those that can win
      // are visited (mode 4); the coupled arm and grids of a few multipliers visit them all (mode 0)
      const bool bracketed = !(cfg->flags & SOAR_FLAG_COUPLED_SCALE) && cfg->n_beta >= kBracketMinBeta &&
                             cfg->beta_step_pct >= 1;
      // the brackets of two E4M3 codes around the Eq. 6 solution lie at multipliers 0.89 .. 1.13 (E4M3 values are
      // at most an eighth apart): a grid from 0.85 to 1.15 or wider holds them whole (mode 4), a shorter one
      // needs the straight-line path to know the grid's ends (mode 5)
      const int half = cfg->n_beta / 2;
      const bool spans = 100 - half * cfg->beta_step_pct <= 85 &&
                         100 + (cfg->n_beta - 1 - half) * cfg->beta_step_pct >= 115;
      const int mode = !single ? (bracketed ? (spans ? 4 : 5) : 0)
                               : ((cfg->flags & SOAR_FLAG_COUPLED_SCALE) ? 2 : (cfg->n_dq <= 2 ? 1 : 3));
      unsigned int g_it = 0;
      for (int t = t_lo; t < t_hi; ++t) {
        const int reverse = t & 1;
        // with the early stop on, any iteration may turn out to be the last one
        const int last = (t == cfg->max_iters - 1) ? 1 : 0;
        const int emit = (may_stop || last) ? 1 : 0;
        const int pg = static_cast<int>(g_last);
        ScopedLaunch sl(K_ITERATE, st);
#define SOAR_LAUNCH_ITERATE(M, D)                                                           \
  do {                                                                                      \
    if (g_it == 0) g_it = persistent_grid(iterate_kernel<M, D>, tiles, kThreads);           \
    iterate_kernel<M, D><<<g_it, kThreads, 0, st>>>(bt, t, reverse, emit, !last, pg);       \
  } while (0)
        if (det) {
          if (mode == 0) SOAR_LAUNCH_ITERATE(0, true);
          else if (mode == 1) SOAR_LAUNCH_ITERATE(1, true);
          else if (mode == 2) SOAR_LAUNCH_ITERATE(2, true);
          else if (mode == 3) SOAR_LAUNCH_ITERATE(3, true);
          else if (mode == 4) SOAR_LAUNCH_ITERATE(4, true);
          else SOAR_LAUNCH_ITERATE(5, true);
        } else {
          if (mode == 0) SOAR_LAUNCH_ITERATE(0, false);
          else if (mode == 1) SOAR_LAUNCH_ITERATE(1, false);
          else if (mode == 2) SOAR_LAUNCH_ITERATE(2, false);
          else if (mode == 3) SOAR_LAUNCH_ITERATE(3, false);
          else if (mode == 4) SOAR_LAUNCH_ITERATE(4, false);
          else SOAR_LAUNCH_ITERATE(5, false);
        }
#undef SOAR_LAUNCH_ITERATE
        g_last = g_it;
      }
    }
    if (!(stages & kStageFinalize)) continue;
    {
      ScopedLaunch sl(K_FINALIZE, st);
      finalize_kernel<<<bt.n, 128, 0, st>>>(bt, rp, static_cast<int>(g_last));
    }
    if (want_sw) {
      for (int j = 0; j < bt.n; ++j) {
        const soar_tensor_desc& d = tensors[first + j];
        const Params& p = bt.t[j];
        const unsigned int rt = static_cast<unsigned int>((d.rows + 127) / 128);
        const unsigned int ct = (p.nbc + 3) / 4;
        const size_t total = static_cast<size_t>(rt) * ct * 512;
        const size_t blocks = (total + 255) / 256;
        const unsigned int grid = static_cast<unsigned int>(blocks < 65535u * 16u ? blocks : 65535u * 16u);
        ScopedLaunch sl(K_SWIZZLE, st);
        swizzle_kernel<<<grid, 256, 0, st>>>(p.scales, static_cast<uint8_t*>(d.out_e4m3_scales_sw),
                                             static_cast<unsigned int>(d.rows), p.nbc, rt, ct);
      }
    }
  }
  return cudaGetLastError() == cudaSuccess ? SOAR_OK : SOAR_ERR_CUDA;
}

}  // namespace

extern "C" {

int soar_quantize_batch(const soar_tensor_desc* tensors, int n, const soar_cfg* cfg, void* workspace,
                        size_t workspace_bytes, void* stream) {
  const int rc = check_cfg(cfg);
  if (rc != SOAR_OK) return rc;
  return run_batch(tensors, n, cfg, workspace, workspace_bytes, stream, kStageAll, 0, cfg->max_iters);
}

int soar_quantize_stage(const soar_tensor_desc* tensors, int n, const soar_cfg* cfg, void* workspace,
                        size_t workspace_bytes, int stage, void* stream) {
  const int rc = check_cfg(cfg);
  if (rc != SOAR_OK) return rc;
  if (stage == SOAR_STAGE_AMAX) return run_batch(tensors, n, cfg, workspace, workspace_bytes, stream, kStageAmax, 0, 0);
  if (stage == SOAR_STAGE_INIT) return run_batch(tensors, n, cfg, workspace, workspace_bytes, stream, kStageInit, 0, 0);
  if (stage == SOAR_STAGE_FINALIZE)
    return run_batch(tensors, n, cfg, workspace, workspace_bytes, stream, kStageFinalize, 0, 0);
  if (stage < 0 || stage >= cfg->max_iters) return SOAR_ERR_INVALID_ARG;
  return run_batch(tensors, n, cfg, workspace, workspace_bytes, stream, kStageIterate, stage, stage + 1);
}

int soar_quantize(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld, const soar_cfg* cfg,
                  void* out_fp4_packed, void* out_e4m3_scales, void* out_e4m3_scales_sw,
                  float* out_global_fp32, void* workspace, size_t workspace_bytes,
                  soar_result* out_result, void* stream) {
  soar_tensor_desc d;
  d.W_bf16 = W_bf16;
  d.rows = rows;
  d.cols = cols;
  d.ld = ld;
  d.out_fp4_packed = out_fp4_packed;
  d.out_e4m3_scales = out_e4m3_scales;
  d.out_e4m3_scales_sw = out_e4m3_scales_sw;
  d.out_global_fp32 = out_global_fp32;
  d.out_result = out_result;
  return soar_quantize_batch(&d, 1, cfg, workspace, workspace_bytes, stream);
}

// Built-in scratch of soar_quantize_static.  In host code the symbol below is only a handle:
// the device address comes from cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char g_static_scratch[SOAR_STATIC_SCRATCH_BYTES];
// the largest accepted matrix needs exactly this much: the header, 8 bytes of state and one scale byte per block
static_assert(kWsFixedBytes + (SOAR_STATIC_MAX_ELEMENTS / 16) * (sizeof(uint2) + 1) == SOAR_STATIC_SCRATCH_BYTES,
              "SOAR_STATIC_SCRATCH_BYTES does not match the workspace of SOAR_STATIC_MAX_ELEMENTS");

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

namespace {
int dequant_error_impl(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld, const float* h,
                       const void* fp4_packed, const void* e4m3_scales, int scale_layout,
                       const float* global_fp32, double* out_sse, double* out_sumsq, void* stream) {
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
  p.ntiles = (p.nblk + kTile - 1) / kTile;
  p.contiguous = (ld == cols) ? 1 : 0;
  if (cudaMemsetAsync(out_sse, 0, sizeof(double), st) != cudaSuccess) return SOAR_ERR_CUDA;
  if (cudaMemsetAsync(out_sumsq, 0, sizeof(double), st) != cudaSuccess) return SOAR_ERR_CUDA;
  {
    ScopedLaunch sl(K_DEQUANT_ERROR, st);
    Batch bt;
    memset(&bt, 0, sizeof(bt));
    bt.n = 1;
    bt.idle_producer = g_idle_producer;
    bt.t[0] = p;
    bt.total_tiles = p.ntiles;
    for (int j = 0; j < kMaxBatch; ++j) bt.tile_end[j] = j == 0 ? p.ntiles : 0xFFFFFFFFu;
    const uint8_t* sc = static_cast<const uint8_t*>(e4m3_scales);
    const int sw = scale_layout == SOAR_SCALES_SWIZZLED ? 1 : 0;
    if (h == nullptr)
      dequant_error_kernel<false><<<persistent_grid(dequant_error_kernel<false>, p.ntiles, kThreads), kThreads, 0,
                                    st>>>(bt, sc, sw, (p.nbc + 3) / 4, global_fp32, nullptr, out_sse, out_sumsq);
    else
      dequant_error_kernel<true><<<persistent_grid(dequant_error_kernel<true>, p.ntiles, kThreads), kThreads, 0,
                                   st>>>(bt, sc, sw, (p.nbc + 3) / 4, global_fp32, h, out_sse, out_sumsq);
  }
  return cudaGetLastError() == cudaSuccess ? SOAR_OK : SOAR_ERR_CUDA;
}
}  // namespace

int soar_dequant_error(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld, const void* fp4_packed,
                       const void* e4m3_scales, int scale_layout, const float* global_fp32,
                       double* out_sse, double* out_sumsq, void* stream) {
  return dequant_error_impl(W_bf16, rows, cols, ld, nullptr, fp4_packed, e4m3_scales, scale_layout, global_fp32,
                            out_sse, out_sumsq, stream);
}

int soar_dequant_error_weighted(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld,
                                const float* col_weight, const void* fp4_packed, const void* e4m3_scales,
                                int scale_layout, const float* global_fp32, double* out_sse,
                                double* out_sumsq, void* stream) {
  if (col_weight == nullptr) return SOAR_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(col_weight) % 16 != 0) return SOAR_ERR_UNSUPPORTED;
  return dequant_error_impl(W_bf16, rows, cols, ld, col_weight, fp4_packed, e4m3_scales, scale_layout,
                            global_fp32, out_sse, out_sumsq, stream);
}

size_t soar_weighted_workspace_bytes(int64_t rows, int64_t cols, const soar_cfg* cfg) {
  if (check_cfg(cfg) != SOAR_OK || rows <= 0 || cols <= 0 || cols % 16 != 0) return 0;
  const size_t nblk = static_cast<size_t>(rows) * static_cast<size_t>(cols / 16);
  size_t n = kWsFixedBytes;
  if (cfg->max_iters > 0) n += round256(nblk * sizeof(double2)) + round256(nblk);
  if (!(cfg->scale_layout & SOAR_SCALES_LINEAR)) n += round256(nblk);
  return n;
}

size_t soar_weighted_batch_workspace_bytes(const soar_tensor_desc* tensors, int n, const soar_cfg* cfg) {
  if (tensors == nullptr || n <= 0) return 0;
  size_t total = 0;
  for (int i = 0; i < n; ++i) {
    const size_t b = soar_weighted_workspace_bytes(tensors[i].rows, tensors[i].cols, cfg);
    if (b == 0) return 0;
    total += b;
  }
  return total;
}

int soar_quantize_weighted_batch(const soar_tensor_desc* tensors, const float* const* col_weights, int n,
                                 const soar_cfg* cfg, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_cfg(cfg);
  if (rc != SOAR_OK) return rc;
  if (cfg->flags & SOAR_FLAG_DETERMINISTIC) return SOAR_ERR_UNSUPPORTED;   // the weighted passes add with atomics only
  if (tensors == nullptr || col_weights == nullptr || n <= 0) return SOAR_ERR_INVALID_ARG;
  const bool want_lin = (cfg->scale_layout & SOAR_SCALES_LINEAR) != 0;
  const bool want_sw = (cfg->scale_layout & SOAR_SCALES_SWIZZLED) != 0;
  for (int i = 0; i < n; ++i) {   // every argument is checked before anything is enqueued
    const soar_tensor_desc& d = tensors[i];
    rc = check_shape(d.W_bf16, d.rows, d.cols, d.ld);
    if (rc != SOAR_OK) return rc;
    if (col_weights[i] == nullptr || d.out_fp4_packed == nullptr || d.out_global_fp32 == nullptr)
      return SOAR_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(col_weights[i]) % 16 != 0 || reinterpret_cast<uintptr_t>(d.out_fp4_packed) % 16 != 0)
      return SOAR_ERR_UNSUPPORTED;
    if (want_lin && d.out_e4m3_scales == nullptr) return SOAR_ERR_INVALID_ARG;
    if (want_sw && d.out_e4m3_scales_sw == nullptr) return SOAR_ERR_INVALID_ARG;
  }
  const size_t need = soar_weighted_batch_workspace_bytes(tensors, n, cfg);
  if (workspace == nullptr || need == 0 || workspace_bytes < need) return SOAR_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return SOAR_ERR_UNSUPPORTED;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // workspace: the n headers first (one memset clears them all), then each tensor's arrays
  uint8_t* const headers = static_cast<uint8_t*>(workspace);
  uint8_t* next = headers + static_cast<size_t>(n) * kWsFixedBytes;
  if (cudaMemsetAsync(headers, 0, static_cast<size_t>(n) * kWsFixedBytes, st) != cudaSuccess) return SOAR_ERR_CUDA;
  const bool may_stop = cfg->early_stop_rel > 0.0f;
  for (int first = 0; first < n; first += kMaxBatch) {
    Batch bt;
    WeightedBatch wb;
    Reports rp;
    memset(&bt, 0, sizeof(bt));
    memset(&wb, 0, sizeof(wb));
    memset(&rp, 0, sizeof(rp));
    bt.n = (n - first < kMaxBatch) ? n - first : kMaxBatch;
    bt.idle_producer = g_idle_producer;
    unsigned int tiles = 0;
    for (int j = 0; j < bt.n; ++j) {
      const soar_tensor_desc& d = tensors[first + j];
      Params& p = bt.t[j];
      Weighted& wq = wb.t[j];
      p.W = static_cast<const uint16_t*>(d.W_bf16);
      p.packed = static_cast<uint8_t*>(d.out_fp4_packed);
      p.ws = reinterpret_cast<Ws*>(headers + static_cast<size_t>(first + j) * kWsFixedBytes);
      p.ld = d.ld;
      p.nbc = static_cast<unsigned int>(d.cols / 16);
      p.nblk = static_cast<unsigned int>(d.rows * (d.cols / 16));
      p.ntiles = (p.nblk + kTile - 1) / kTile;
      p.contiguous = (d.ld == d.cols) ? 1 : 0;
      wq.h = col_weights[first + j];
      if (cfg->max_iters > 0) {
        wq.sums = reinterpret_cast<double2*>(next);
        next += round256(static_cast<size_t>(p.nblk) * sizeof(double2));
        wq.code = next;
        next += round256(p.nblk);
      }
      if (want_lin) {
        p.scales = static_cast<uint8_t*>(d.out_e4m3_scales);
      } else {
        p.scales = next;
        next += round256(p.nblk);
      }
      p.max_iters = cfg->max_iters;
      p.early_stop_rel = cfg->early_stop_rel;
      p.n_dq = cfg->n_dq;
      p.n_beta = cfg->n_beta;
      p.beta_step_pct = cfg->beta_step_pct;
      p.flags = cfg->flags;
      tiles += p.ntiles;
      bt.tile_end[j] = tiles;
      rp.alpha[j] = d.out_global_fp32;
      rp.result[j] = d.out_result;
    }
    for (int j = bt.n; j < kMaxBatch; ++j) bt.tile_end[j] = 0xFFFFFFFFu;   // never reached by a tile index
    bt.total_tiles = tiles;

    int reverse = 1;   // the first pass runs forward; each later one starts where the last ended
    {
      ScopedLaunch sl(K_WEIGHTED_AMAX, st);
      weighted_amax_kernel<<<persistent_grid(weighted_amax_kernel, tiles, kThreads), kThreads, 0, st>>>(bt, wb);
    }
    {
      ScopedLaunch sl(K_WEIGHTED_INIT, st);
      weighted_init_kernel<<<persistent_grid(weighted_init_kernel, tiles, kThreads), kThreads, 0, st>>>(
          bt, wb, reverse, cfg->max_iters == 0 ? 1 : 0);
    }
    const unsigned int g_it = persistent_grid(weighted_iterate_kernel, tiles, kThreads);
    for (int t = 0; t < cfg->max_iters; ++t) {
      reverse ^= 1;
      const int last = (t == cfg->max_iters - 1) ? 1 : 0;
      ScopedLaunch sl(K_WEIGHTED_ITERATE, st);
      weighted_iterate_kernel<<<g_it, kThreads, 0, st>>>(bt, wb, t, reverse, (may_stop || last) ? 1 : 0, !last);
    }
    {
      ScopedLaunch sl(K_FINALIZE, st);
      finalize_kernel<<<bt.n, 128, 0, st>>>(bt, rp, 0);
    }
    if (want_sw) {
      for (int j = 0; j < bt.n; ++j) {
        const soar_tensor_desc& d = tensors[first + j];
        const Params& p = bt.t[j];
        const unsigned int rt = static_cast<unsigned int>((d.rows + 127) / 128);
        const unsigned int ct = (p.nbc + 3) / 4;
        const size_t blocks = (static_cast<size_t>(rt) * ct * 512 + 255) / 256;
        const unsigned int grid = static_cast<unsigned int>(blocks < 65535u * 16u ? blocks : 65535u * 16u);
        ScopedLaunch sl(K_SWIZZLE, st);
        swizzle_kernel<<<grid, 256, 0, st>>>(p.scales, static_cast<uint8_t*>(d.out_e4m3_scales_sw),
                                             static_cast<unsigned int>(d.rows), p.nbc, rt, ct);
      }
    }
  }
  return cudaGetLastError() == cudaSuccess ? SOAR_OK : SOAR_ERR_CUDA;
}

int soar_quantize_weighted(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld, const float* col_weight,
                           const soar_cfg* cfg, void* out_fp4_packed, void* out_e4m3_scales,
                           void* out_e4m3_scales_sw, float* out_global_fp32, void* workspace,
                           size_t workspace_bytes, soar_result* out_result, void* stream) {
  soar_tensor_desc d;
  d.W_bf16 = W_bf16;
  d.rows = rows;
  d.cols = cols;
  d.ld = ld;
  d.out_fp4_packed = out_fp4_packed;
  d.out_e4m3_scales = out_e4m3_scales;
  d.out_e4m3_scales_sw = out_e4m3_scales_sw;
  d.out_global_fp32 = out_global_fp32;
  d.out_result = out_result;
  return soar_quantize_weighted_batch(&d, &col_weight, 1, cfg, workspace, workspace_bytes, stream);
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
  // every check soar_quantize would make on the staging buffers, before anything is enqueued
  rc = check_shape(dev->W, rows, cols, ld);
  if (rc != SOAR_OK) return rc;
  if (reinterpret_cast<uintptr_t>(dev->packed) % 16 != 0) return SOAR_ERR_UNSUPPORTED;
  const size_t need = soar_workspace_bytes(rows, cols, cfg);
  if (dev->workspace == nullptr || need == 0 || dev->workspace_bytes < need) return SOAR_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(dev->workspace) % 256 != 0) return SOAR_ERR_UNSUPPORTED;
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

}  // extern "C"

// Host bookkeeping of a pipeline: the slots, three events per slot, the streams and whose turn it is.
struct soar_pipeline {
  std::vector<soar_slot> slots;
  std::vector<cudaEvent_t> loaded, computed, stored;   // per slot: input landed, quantized, results left
  cudaStream_t h2d, compute, d2h;
  size_t next;
};

namespace {
void release_events(soar_pipeline* p) {
  for (cudaEvent_t e : p->loaded) cudaEventDestroy(e);
  for (cudaEvent_t e : p->computed) cudaEventDestroy(e);
  for (cudaEvent_t e : p->stored) cudaEventDestroy(e);
}

// Every rule a matrix must meet to go through slot `sl` (nothing is enqueued before all matrices pass).
int check_host_matrix(const soar_host_matrix& m, const soar_slot& sl, const soar_cfg* cfg, bool weighted) {
  if (m.W_host == nullptr || m.out_fp4_packed_host == nullptr || m.out_global_host == nullptr)
    return SOAR_ERR_INVALID_ARG;
  int rc = check_shape(sl.dev.W, m.rows, m.cols, m.ld);
  if (rc != SOAR_OK) return rc;
  const bool want_lin = (cfg->scale_layout & SOAR_SCALES_LINEAR) != 0;
  const bool want_sw = (cfg->scale_layout & SOAR_SCALES_SWIZZLED) != 0;
  if (want_lin && (m.out_e4m3_scales_host == nullptr || sl.dev.scales == nullptr)) return SOAR_ERR_INVALID_ARG;
  if (want_sw && (m.out_e4m3_scales_sw_host == nullptr || sl.dev.scales_sw == nullptr)) return SOAR_ERR_INVALID_ARG;
  if (m.out_result_host != nullptr && sl.dev.result == nullptr) return SOAR_ERR_INVALID_ARG;
  const size_t n = static_cast<size_t>(m.rows) * static_cast<size_t>(m.cols);
  if (static_cast<size_t>(m.rows) * static_cast<size_t>(m.ld) * 2 > sl.W_bytes || n / 2 > sl.packed_bytes)
    return SOAR_ERR_TOO_LARGE;
  if (want_lin && n / 16 > sl.scales_bytes) return SOAR_ERR_TOO_LARGE;
  if (want_sw && soar_swizzled_scale_bytes(m.rows, m.cols) > sl.scales_sw_bytes) return SOAR_ERR_TOO_LARGE;
  const size_t need = weighted ? soar_weighted_workspace_bytes(m.rows, m.cols, cfg)
                               : soar_workspace_bytes(m.rows, m.cols, cfg);
  if (need == 0 || sl.dev.workspace_bytes < need) return SOAR_ERR_WORKSPACE;
  return SOAR_OK;
}
}  // namespace

extern "C" {

int soar_pipeline_create(soar_pipeline** out, const soar_slot* slots, int n_slots, void* stream_h2d,
                         void* stream_compute, void* stream_d2h) {
  if (out == nullptr || slots == nullptr || n_slots < 1) return SOAR_ERR_INVALID_ARG;
  if (stream_h2d == stream_compute || stream_compute == stream_d2h || stream_h2d == stream_d2h)
    return SOAR_ERR_INVALID_ARG;
  for (int i = 0; i < n_slots; ++i) {
    const soar_staging& d = slots[i].dev;
    if (d.W == nullptr || d.packed == nullptr || d.alpha == nullptr || d.workspace == nullptr)
      return SOAR_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d.W) % 16 != 0 || reinterpret_cast<uintptr_t>(d.packed) % 16 != 0 ||
        reinterpret_cast<uintptr_t>(d.workspace) % 256 != 0)
      return SOAR_ERR_UNSUPPORTED;
  }
  soar_pipeline* p = new (std::nothrow) soar_pipeline();
  if (p == nullptr) return SOAR_ERR_INVALID_ARG;
  p->slots.assign(slots, slots + n_slots);
  p->h2d = static_cast<cudaStream_t>(stream_h2d);
  p->compute = static_cast<cudaStream_t>(stream_compute);
  p->d2h = static_cast<cudaStream_t>(stream_d2h);
  p->next = 0;
  bool ok = true;
  for (int i = 0; i < 3 * n_slots && ok; ++i) {
    cudaEvent_t e;
    ok = cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
    if (ok) (i % 3 == 0 ? p->loaded : i % 3 == 1 ? p->computed : p->stored).push_back(e);
  }
  // a slot is free from the start: its "results left" event is recorded once on the third stream
  for (size_t i = 0; i < p->stored.size() && ok; ++i) ok = cudaEventRecord(p->stored[i], p->d2h) == cudaSuccess;
  if (!ok || p->stored.size() != static_cast<size_t>(n_slots)) {
    release_events(p);
    delete p;
    return SOAR_ERR_CUDA;
  }
  *out = p;
  return SOAR_OK;
}

int soar_pipeline_run(soar_pipeline* pipe, const soar_host_matrix* mats, int n, const soar_cfg* cfg,
                      const float* const* col_weights) {
  if (pipe == nullptr || mats == nullptr || n < 0) return SOAR_ERR_INVALID_ARG;
  int rc = check_cfg(cfg);
  if (rc != SOAR_OK) return rc;
  const size_t ns = pipe->slots.size();
  for (int i = 0; i < n; ++i) {   // everything is checked before anything is enqueued
    const float* h = col_weights != nullptr ? col_weights[i] : nullptr;
    if (h != nullptr && reinterpret_cast<uintptr_t>(h) % 16 != 0) return SOAR_ERR_UNSUPPORTED;
    rc = check_host_matrix(mats[i], pipe->slots[(pipe->next + static_cast<size_t>(i)) % ns], cfg, h != nullptr);
    if (rc != SOAR_OK) return rc;
  }
  const bool want_lin = (cfg->scale_layout & SOAR_SCALES_LINEAR) != 0;
  const bool want_sw = (cfg->scale_layout & SOAR_SCALES_SWIZZLED) != 0;
  for (int i = 0; i < n; ++i) {
    const soar_host_matrix& m = mats[i];
    const size_t si = pipe->next % ns;
    ++pipe->next;
    const soar_staging& d = pipe->slots[si].dev;
    const float* h = col_weights != nullptr ? col_weights[i] : nullptr;
    // copy in, once the slot's previous results have left
    bool ok = cudaStreamWaitEvent(pipe->h2d, pipe->stored[si], 0) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(d.W, m.W_host, static_cast<size_t>(m.rows) * static_cast<size_t>(m.ld) * 2,
                               cudaMemcpyHostToDevice, pipe->h2d) == cudaSuccess;
    ok = ok && cudaEventRecord(pipe->loaded[si], pipe->h2d) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(pipe->compute, pipe->loaded[si], 0) == cudaSuccess;
    if (!ok) return SOAR_ERR_CUDA;
    soar_result* res = m.out_result_host != nullptr ? d.result : nullptr;
    rc = h == nullptr ? soar_quantize(d.W, m.rows, m.cols, m.ld, cfg, d.packed, d.scales, d.scales_sw, d.alpha,
                                      d.workspace, d.workspace_bytes, res, pipe->compute)
                      : soar_quantize_weighted(d.W, m.rows, m.cols, m.ld, h, cfg, d.packed, d.scales, d.scales_sw,
                                               d.alpha, d.workspace, d.workspace_bytes, res, pipe->compute);
    if (rc != SOAR_OK) return rc;
    ok = cudaEventRecord(pipe->computed[si], pipe->compute) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(pipe->d2h, pipe->computed[si], 0) == cudaSuccess;
    const size_t ne = static_cast<size_t>(m.rows) * static_cast<size_t>(m.cols);
    ok = ok && cudaMemcpyAsync(m.out_fp4_packed_host, d.packed, ne / 2, cudaMemcpyDeviceToHost, pipe->d2h) ==
                   cudaSuccess;
    if (want_lin)
      ok = ok && cudaMemcpyAsync(m.out_e4m3_scales_host, d.scales, ne / 16, cudaMemcpyDeviceToHost, pipe->d2h) ==
                     cudaSuccess;
    if (want_sw)
      ok = ok && cudaMemcpyAsync(m.out_e4m3_scales_sw_host, d.scales_sw, soar_swizzled_scale_bytes(m.rows, m.cols),
                                 cudaMemcpyDeviceToHost, pipe->d2h) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(m.out_global_host, d.alpha, sizeof(float), cudaMemcpyDeviceToHost, pipe->d2h) ==
                   cudaSuccess;
    if (res != nullptr)
      ok = ok && cudaMemcpyAsync(m.out_result_host, d.result, sizeof(soar_result), cudaMemcpyDeviceToHost,
                                 pipe->d2h) == cudaSuccess;
    ok = ok && cudaEventRecord(pipe->stored[si], pipe->d2h) == cudaSuccess;
    if (!ok) return SOAR_ERR_CUDA;
  }
  return SOAR_OK;
}

int soar_pipeline_synchronize(soar_pipeline* pipe) {
  if (pipe == nullptr) return SOAR_ERR_INVALID_ARG;
  return cudaStreamSynchronize(pipe->d2h) == cudaSuccess ? SOAR_OK : SOAR_ERR_CUDA;
}

void soar_pipeline_destroy(soar_pipeline* pipe) {
  if (pipe == nullptr) return;
  cudaStreamSynchronize(pipe->h2d);
  cudaStreamSynchronize(pipe->compute);
  cudaStreamSynchronize(pipe->d2h);
  release_events(pipe);
  delete pipe;
}

int soar_selftest_reciprocal(int lo_exp, int hi_exp, unsigned long long* out_mismatches, void* stream) {
  if (out_mismatches == nullptr || lo_exp < 2 || hi_exp > 252 || lo_exp > hi_exp) return SOAR_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(out_mismatches, 0, sizeof(unsigned long long), st) != cudaSuccess) return SOAR_ERR_CUDA;
  selftest_reciprocal_kernel<<<sm_count() * 8, 256, 0, st>>>(static_cast<unsigned int>(lo_exp),
                                                             static_cast<unsigned int>(hi_exp), out_mismatches);
  return cudaGetLastError() == cudaSuccess ? SOAR_OK : SOAR_ERR_CUDA;
}

int soar_mx_quantize(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld, int n_dq, int n_beta,
                     int beta_step_pct, void* out_fp4_packed, void* out_e8m0_scales, soar_mx_result* out_result,
                     void* stream) {
  const int rc = check_shape(W_bf16, rows, cols, ld);
  if (rc != SOAR_OK) return rc;
  if (cols % 32 != 0) return SOAR_ERR_UNSUPPORTED;
  if (out_fp4_packed == nullptr || out_e8m0_scales == nullptr || out_result == nullptr) return SOAR_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(out_fp4_packed) % 16 != 0 || reinterpret_cast<uintptr_t>(out_result) % 8 != 0)
    return SOAR_ERR_UNSUPPORTED;
  if (n_beta < 0 || n_beta > SOAR_MAX_BETA || n_dq < 1 || n_dq > SOAR_MAX_DQ || beta_step_pct < 0)
    return SOAR_ERR_INVALID_ARG;
  if (n_beta > 0 && 100 - (n_beta / 2) * beta_step_pct <= 0) return SOAR_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(out_result, 0, sizeof(soar_mx_result), st) != cudaSuccess) return SOAR_ERR_CUDA;
  Batch bt;
  memset(&bt, 0, sizeof(bt));
  Params& p = bt.t[0];
  p.W = static_cast<const uint16_t*>(W_bf16);
  p.packed = static_cast<uint8_t*>(out_fp4_packed);
  p.ld = ld;
  p.nbc = static_cast<unsigned int>(cols / 16);
  p.nblk = static_cast<unsigned int>(rows * (cols / 16));
  p.ntiles = (p.nblk + kTile - 1) / kTile;
  p.contiguous = (ld == cols) ? 1 : 0;
  bt.n = 1;
  bt.idle_producer = g_idle_producer;
  bt.total_tiles = p.ntiles;
  for (int j = 0; j < kMaxBatch; ++j) bt.tile_end[j] = j == 0 ? p.ntiles : 0xFFFFFFFFu;
  uint8_t* sc = static_cast<uint8_t*>(out_e8m0_scales);
  double* gsum = &out_result->reserved;   // the running sum of the blocks' errors minus sum W^2
  {
    ScopedLaunch sl(K_MX, st);
    if (n_beta == 0)
      mx_kernel<false><<<persistent_grid(mx_kernel<false>, p.ntiles, kThreads), kThreads, 0, st>>>(
          bt, sc, out_result, gsum, n_dq, n_beta, beta_step_pct);
    else
      mx_kernel<true><<<persistent_grid(mx_kernel<true>, p.ntiles, kThreads), kThreads, 0, st>>>(
          bt, sc, out_result, gsum, n_dq, n_beta, beta_step_pct);
  }
  mx_finalize_kernel<<<1, 1, 0, st>>>(out_result, gsum);
  return cudaGetLastError() == cudaSuccess ? SOAR_OK : SOAR_ERR_CUDA;
}

int soar_debug_fail_waits(int on) {
  g_idle_producer = on ? 1 : 0;
  return SOAR_OK;
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
    case SOAR_ERR_TOO_LARGE: return "matrix exceeds the built-in scratch of soar_quantize_static or a pipeline slot";
    default: return "unknown status";
  }
}

}  // extern "C"
