// Separable transform on the tensor cores ("Separable spectral decomposition", "Reconstruction"),
// bf16 storage, head_dim 128.  Every axis pass is the same batched contraction: for one line of n
// grid positions along the axis (all other coordinates fixed),
//     D[c][a] = sum_b X[b][c] * Mat[a][b]          c = channel (128), a = output index, b = input index
// The data tile X (n rows of 128 channels, 256 bytes each) is the A operand, taken straight from a
// TMA box in shared memory as an MN-major matrix (M = channels), the transform matrix is the
// K-major B operand, and the 128 x n fp32 result sits in tensor memory with one channel per lane.
// Precision: the transform matrix is split into bf16 hi + lo parts, and so is every intermediate
// between two axis passes (two bf16 grids, hi = bf16(v), lo = bf16(v - hi)); a pass then issues
// X_hi*C_hi + X_hi*C_lo + X_lo*C_hi per k-step.  Intermediates can be far larger than the final
// values (low-frequency content, the constant offset the exchange adds to a whole band), so a
// single bf16 rounding between passes would not meet the output tolerance.
//
// A CTA is persistent over "stages" of LPS consecutive lines (LPS * n = 128 rows; 32 KB of bf16
// input, or 64 KB when the input is a hi/lo pair).
//   warp 0      TMA producer (ring of 2-4 stages, as many as fit beside the matrix images)
//   warp 1      tcgen05.mma issuer, 4 accumulator buffers of 128 TMEM columns
//   warps 2..5  epilogue: tcgen05.ld, convert, store (thread = channel, so a warp writes 32
//               consecutive channels of one output position per instruction)
// Modes: FIRST  caller's Q/K/V -> hi/lo intermediate, plus an fp32 copy of the columns k_w < L_w
//               from which the low band is computed at full precision
//        MIDDLE intermediate (hi/lo, or a single bf16 grid) -> hi/lo intermediate
//        SPLIT  intermediate -> band-major mid/high coefficient buffers (rank evaluated in
//               registers) with the router's band energies accumulated from the fp32 accumulators
//        LAST   intermediate -> the caller's out tensor
#include <cuda.h>

#include "ff_internal.h"
#include "ff_sm100.cuh"

using namespace sm100;

namespace {

constexpr int CH = 128;
constexpr int STAGE_ROWS = 128;
constexpr int TILE_BYTES = STAGE_ROWS * CH * 2;    // 32 KB: 128 rows of bf16
constexpr int MAX_STAGE = 4;
constexpr int NACC = 4;
constexpr int DCT_TC_THREADS = 192;

enum { MODE_FIRST = 0, MODE_MIDDLE = 1, MODE_SPLIT = 2, MODE_LAST = 3 };

struct DctTcParams {
  FFDims dm;
  const float* mat;        // [n][n] fp32, out[a] = sum_b mat[a][b] in[b]
  int n;                   // axis length
  int axis;                // 0 = t, 1 = h, 2 = w
  int mode;
  int group;               // tensor-heads in this launch
  int group_start;         // index of the first one (tensor * BH + bh for the forward, bh for the inverse)
  int lines_per_th;        // lines per tensor-head = N / n
  int in_split;            // input is a hi/lo pair of grids (map0 = hi, map1 = lo)
  int nstage;              // ring depth
  __nv_bfloat16* dst;      // hi grid [group][T][H][W][128], or the out tensor (MODE_LAST)
  __nv_bfloat16* dst_lo;   // lo grid
  float* side;             // MODE_FIRST: [group][T][H][L_w][128] fp32
  __nv_bfloat16* spec_mid; __nv_bfloat16* spec_high;
  double* energy;          // [B][3][128]
  int* status;
};

struct DctShared {
  uint64_t full[MAX_STAGE], empty[MAX_STAGE], acc_full[NACC], acc_empty[NACC];
  uint32_t tmem_base;
  int abort_flag;
};

// Coordinates (w, h, t) of the first position of line `line` of a tensor-head, for the given axis.
__device__ __forceinline__ void line_origin(const FFDims& dm, int axis, int line, int& w, int& h, int& t) {
  if (axis == 2) { w = 0; h = line % dm.H; t = line / dm.H; }
  else if (axis == 1) { h = 0; w = line % dm.W; t = line / dm.W; }
  else { t = 0; w = line % dm.W; h = line / dm.W; }
}

__device__ __forceinline__ void tma_load_5d(void* smem_dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2,
                                            int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

// Three source maps (Q, K, V) in MODE_FIRST; otherwise map0 (= hi) and, for split input, map1 (= lo).
__global__ void __launch_bounds__(DCT_TC_THREADS, 1)
dct_tc_kernel(const __grid_constant__ CUtensorMap map0, const __grid_constant__ CUtensorMap map1,
              const __grid_constant__ CUtensorMap map2, const DctTcParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const FFDims& dm = P.dm;
  const int n = P.n;
  const int NSTAGE = P.nstage;
  const int STAGE_BYTES = P.in_split ? 2 * TILE_BYTES : TILE_BYTES;
  const int img_bytes = (n > 64 ? 2 : 1) * n * 128;       // one matrix image
  uint8_t* sData = smem;                                  // NSTAGE x STAGE_BYTES
  uint8_t* sHi = smem + NSTAGE * STAGE_BYTES;             // basis hi: [half][n rows][128 B], swizzled
  uint8_t* sLo = sHi + img_bytes;                         // basis lo
  DctShared& sh = *(DctShared*)(sLo + img_bytes);
  const int lps = STAGE_ROWS / n;                         // lines per stage
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_lines = P.group * P.lines_per_th;
  const int total_stages = (total_lines + lps - 1) / lps;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NSTAGE; ++i) { mbar_init(&sh.full[i], 1); mbar_init(&sh.empty[i], 1); }
    for (int i = 0; i < NACC; ++i) { mbar_init(&sh.acc_full[i], 1); mbar_init(&sh.acc_empty[i], 128); }
    sh.abort_flag = 0;
    fence_mbar_init();
  }
  // Transform matrix as the K-major B operand: row a = output index, 64 input indices per 128-byte
  // row, 16-byte chunks XOR-swizzled with the row index (the 128-byte swizzle the MMA expects).
  for (int idx = threadIdx.x; idx < n * n; idx += DCT_TC_THREADS) {
    const int a = idx / n, b = idx % n;
    const float v = P.mat[idx];
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    const __nv_bfloat16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
    const int half = b >> 6, bk = b & 63;
    const uint32_t off = half * (n * 128) + a * 128 + ((((bk >> 3) ^ (a & 7)) << 4) | ((bk & 7) << 1));
    *(__nv_bfloat16*)(sHi + off) = hi;
    *(__nv_bfloat16*)(sLo + off) = lo;
  }
  fence_proxy_async();                                    // generic-proxy writes -> visible to the MMA's async proxy
  if (warp == 1) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = sh.tmem_base;
  volatile int* abort_flag = &sh.abort_flag;
  const int half_stride = lps * n * 128;                  // bytes between the two 64-channel halves of a stage (= 16 KB)

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_desc(&map0);
      unsigned it = 0;
      bool ok = true;
      for (int s = blockIdx.x; s < total_stages && ok; s += gridDim.x, ++it) {
        const int slot = it % NSTAGE;
        if (it >= NSTAGE) ok = mbar_wait(&sh.empty[slot], ((it / NSTAGE) - 1) & 1, abort_flag);
        if (!ok) break;
        uint8_t* dst = sData + slot * STAGE_BYTES;
        int nl = total_lines - s * lps; if (nl > lps) nl = lps;
        mbar_arrive_expect_tx(&sh.full[slot], nl * n * 256 * (P.in_split ? 2 : 1));
        for (int l = 0; l < nl; ++l) {
          const int gl = s * lps + l;
          const int gi = gl / P.lines_per_th, line = gl % P.lines_per_th;
          int w, h, t; line_origin(dm, P.axis, line, w, h, t);
          const CUtensorMap* map = &map0;
          int slice = gi;
          if (P.mode == MODE_FIRST) {
            const int th = P.group_start + gi;
            const int tensor = th / dm.BH;
            map = tensor == 0 ? &map0 : (tensor == 1 ? &map1 : &map2);
            slice = th % dm.BH;
          }
          tma_load_5d(dst + l * n * 128, map, &sh.full[slot], 0, w, h, t, slice);
          tma_load_5d(dst + half_stride + l * n * 128, map, &sh.full[slot], 64, w, h, t, slice);
          if (P.in_split) {
            tma_load_5d(dst + TILE_BYTES + l * n * 128, &map1, &sh.full[slot], 0, w, h, t, slice);
            tma_load_5d(dst + TILE_BYTES + half_stride + l * n * 128, &map1, &sh.full[slot], 64, w, h, t, slice);
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(CH, n, /*a_mn_major=*/true, /*b_mn_major=*/false);
      unsigned it = 0;
      bool ok = true;
      for (int s = blockIdx.x; s < total_stages && ok; s += gridDim.x, ++it) {
        const int slot = it % NSTAGE, ab = it % NACC;
        ok = mbar_wait(&sh.full[slot], (it / NSTAGE) & 1, abort_flag);
        if (ok && it >= NACC) ok = mbar_wait(&sh.acc_empty[ab], ((it / NACC) - 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        int nl = total_lines - s * lps; if (nl > lps) nl = lps;
        const uint32_t dbase = smem_u32(sData + slot * STAGE_BYTES);
        for (int l = 0; l < nl; ++l) {
          const uint32_t d_tm = tm + ab * 128 + l * n;
          for (int ks = 0; ks < n / 16; ++ks) {
            const uint64_t adesc = smem_desc_sw128(dbase + l * n * 128 + ks * 2048, half_stride, 1024);
            const uint32_t boff = (ks >> 2) * (n * 128) + (ks & 3) * 32;
            const uint64_t bhi = smem_desc_sw128(smem_u32(sHi) + boff, 16, 1024);
            umma_ss(d_tm, adesc, bhi, idesc, ks > 0 ? 1u : 0u);
            umma_ss(d_tm, adesc, smem_desc_sw128(smem_u32(sLo) + boff, 16, 1024), idesc, 1u);
            if (P.in_split)
              umma_ss(d_tm, smem_desc_sw128(dbase + TILE_BYTES + l * n * 128 + ks * 2048, half_stride, 1024), bhi, idesc, 1u);
          }
        }
        umma_commit(&sh.empty[slot]);
        umma_commit(&sh.acc_full[ab]);
      }
    }
  } else {
    const int quarter = warp & 3;
    const int c = quarter * 32 + lane;                    // channel of this thread
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const long long N_d = dm.N * CH;
    const long long axis_stride = (P.axis == 2 ? 1LL : (P.axis == 1 ? (long long)dm.W : (long long)dm.W * dm.H)) * CH;
    float e_mid = 0.f, e_high = 0.f;
    int e_sample = -1;
    unsigned it = 0;
    bool ok = true;
    for (int s = blockIdx.x; s < total_stages && ok; s += gridDim.x, ++it) {
      const int ab = it % NACC;
      ok = __all_sync(0xffffffffu, mbar_wait(&sh.acc_full[ab], (it / NACC) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      int nl = total_lines - s * lps; if (nl > lps) nl = lps;
      for (int l = 0; l < nl; ++l) {
        const int gl = s * lps + l;
        const int gi = gl / P.lines_per_th, line = gl % P.lines_per_th;
        int w, h, t; line_origin(dm, P.axis, line, w, h, t);
        const long long pos0 = (((long long)t * dm.H + h) * dm.W + w) * CH + c;     // first position of the line
        const int th = P.group_start + gi;
        if (P.mode == MODE_SPLIT) {
          const int sample = (th % dm.BH) / dm.heads;
          if (sample != e_sample) {
            if (e_sample >= 0 && P.energy) {
              atomicAdd(P.energy + ((size_t)e_sample * 3 + 1) * CH + c, (double)e_mid);
              atomicAdd(P.energy + ((size_t)e_sample * 3 + 2) * CH + c, (double)e_high);
            }
            e_mid = e_high = 0.f; e_sample = sample;
          }
        }
        for (int a0 = 0; a0 < n; a0 += 16) {
          uint32_t r[16];
          tmem_ld16(tm + lane_addr + ab * 128 + l * n + a0, r);
          tmem_wait_ld();
          if (P.mode == MODE_SPLIT) {
            // Band and rank of (k_t, h, w) for k_t = a0 .. a0+15 from per-line constants: along k_t
            // the counts of box members below the coefficient are piecewise linear.
            const int tensor = th / dm.BH, bh = th % dm.BH;
            const bool hw_low = h < dm.L[1] && w < dm.L[2], hw_mid = h < dm.M[1] && w < dm.M[2];
            const int Lhw = dm.L[1] * dm.L[2], Mhw = dm.M[1] * dm.M[2];
            const int offL = (h < dm.L[1] ? h : dm.L[1]) * dm.L[2] + (h < dm.L[1] ? (w < dm.L[2] ? w : dm.L[2]) : 0);
            const int offM = (h < dm.M[1] ? h : dm.M[1]) * dm.M[2] + (h < dm.M[1] ? (w < dm.M[2] ? w : dm.M[2]) : 0);
            __nv_bfloat16* mid_base = P.spec_mid + ((size_t)tensor * dm.BH + bh) * dm.Nmid * CH + c;
            __nv_bfloat16* high_base = P.spec_high + ((size_t)tensor * dm.BH + bh) * dm.Nhigh * CH + c;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float v = __uint_as_float(r[i]);
              const int kt = a0 + i;
              const long long cl = kt < dm.L[0] ? (long long)kt * Lhw + offL : dm.Nlow;
              const long long cm = kt < dm.M[0] ? (long long)kt * Mhw + offM : (long long)dm.M[0] * Mhw;
              if (kt < dm.L[0] && hw_low) continue;                                   // low band: fp32 path
              if (kt < dm.M[0] && hw_mid) {
                mid_base[(cm - cl) * CH] = __float2bfloat16_rn(v);
                e_mid = fmaf(v, v, e_mid);
              } else {
                high_base[((((long long)kt * dm.H + h) * dm.W + w) - cm) * CH] = __float2bfloat16_rn(v);
                e_high = fmaf(v, v, e_high);
              }
            }
          } else {
            const size_t o0 = (size_t)(P.mode == MODE_LAST ? th : gi) * N_d + pos0 + (long long)a0 * axis_stride;
            __nv_bfloat16* dst = P.dst + o0;
            if (P.mode == MODE_LAST) {
#pragma unroll
              for (int i = 0; i < 16; ++i) dst[(long long)i * axis_stride] = __float2bfloat16_rn(__uint_as_float(r[i]));
            } else {
              __nv_bfloat16* dlo = P.dst_lo + o0;
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const float v = __uint_as_float(r[i]);
                const __nv_bfloat16 hi = __float2bfloat16_rn(v);
                dst[(long long)i * axis_stride] = hi;
                dlo[(long long)i * axis_stride] = __float2bfloat16_rn(v - __bfloat162float(hi));
              }
            }
            if (P.mode == MODE_FIRST && a0 < dm.L[2]) {
              float* sd = P.side + ((((size_t)gi * dm.T + t) * dm.H + h) * dm.L[2]) * CH + c;
#pragma unroll
              for (int i = 0; i < 16; ++i)
                if (a0 + i < dm.L[2]) sd[(size_t)(a0 + i) * CH] = __uint_as_float(r[i]);
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(&sh.acc_empty[ab]);
    }
    if (P.mode == MODE_SPLIT && e_sample >= 0 && P.energy) {
      atomicAdd(P.energy + ((size_t)e_sample * 3 + 1) * CH + c, (double)e_mid);
      atomicAdd(P.energy + ((size_t)e_sample * 3 + 2) * CH + c, (double)e_high);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (sh.abort_flag) {
    if (threadIdx.x == 0) atomicExch(P.status, FF_ERR_TIMEOUT);
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tm, 512);
  }
}

// Low band at full precision from the fp32 copy of the w-transformed columns k_w < L_w:
//   low[k_t][k_h][k_w][c] = sum_t C_T[k_t][t] sum_h C_H[k_h][h] side[t][h][k_w][c]
// One CTA per (tensor-head, k_h, k_w); thread = (t group, channel); the t groups are combined through
// shared memory.  Also accumulates the low band's energy.
constexpr int LOW_MAX_LT = 16;
constexpr int LOW_TG = 8;

__global__ void __launch_bounds__(CH * LOW_TG) low_band_kernel(const float* side, const float* CT, const float* CHm,
                                                               float* spec_low, double* energy, FFDims dm, int group_start) {
  const int kw = blockIdx.x % dm.L[2], kh = blockIdx.x / dm.L[2];
  const int gi = blockIdx.y, th = group_start + gi;
  const int c = threadIdx.x % CH, tg = threadIdx.x / CH;
  __shared__ float ch_row[128];
  __shared__ float red[LOW_MAX_LT][CH];
  for (int i = threadIdx.x; i < dm.H; i += CH * LOW_TG) ch_row[i] = CHm[(size_t)kh * dm.H + i];
  float e = 0.f;
  for (int kt0 = 0; kt0 < dm.L[0]; kt0 += LOW_MAX_LT) {
    for (int i = threadIdx.x; i < LOW_MAX_LT * CH; i += CH * LOW_TG) red[i / CH][i % CH] = 0.f;
    __syncthreads();
    float acc[LOW_MAX_LT];
#pragma unroll
    for (int i = 0; i < LOW_MAX_LT; ++i) acc[i] = 0.f;
    for (int t = tg; t < dm.T; t += LOW_TG) {
      const float* col = side + ((((size_t)gi * dm.T + t) * dm.H) * dm.L[2] + kw) * CH + c;
      float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
      int h = 0;
      for (; h + 3 < dm.H; h += 4) {
        s0 = fmaf(ch_row[h], col[(size_t)h * dm.L[2] * CH], s0);
        s1 = fmaf(ch_row[h + 1], col[(size_t)(h + 1) * dm.L[2] * CH], s1);
        s2 = fmaf(ch_row[h + 2], col[(size_t)(h + 2) * dm.L[2] * CH], s2);
        s3 = fmaf(ch_row[h + 3], col[(size_t)(h + 3) * dm.L[2] * CH], s3);
      }
      for (; h < dm.H; ++h) s0 = fmaf(ch_row[h], col[(size_t)h * dm.L[2] * CH], s0);
      const float sh_ = (s0 + s1) + (s2 + s3);
#pragma unroll
      for (int i = 0; i < LOW_MAX_LT; ++i)
        if (kt0 + i < dm.L[0]) acc[i] = fmaf(CT[(size_t)(kt0 + i) * dm.T + t], sh_, acc[i]);
    }
#pragma unroll
    for (int i = 0; i < LOW_MAX_LT; ++i)
      if (kt0 + i < dm.L[0]) atomicAdd(&red[i][c], acc[i]);
    __syncthreads();
    if (tg == 0) {
#pragma unroll
      for (int i = 0; i < LOW_MAX_LT; ++i) {
        if (kt0 + i >= dm.L[0]) break;
        const long long rank = ((long long)(kt0 + i) * dm.L[1] + kh) * dm.L[2] + kw;
        const float v = red[i][c];
        spec_low[((size_t)th * dm.Nlow + rank) * CH + c] = v;
        e = fmaf(v, v, e);
      }
    }
    __syncthreads();
  }
  if (energy && tg == 0) atomicAdd(energy + ((size_t)((th % dm.BH) / dm.heads) * 3) * CH + c, (double)e);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 5-D map over a [slices][T][H][W][128] bf16 grid whose box is one line along `axis`.
bool encode_grid_map(CUtensorMap* map, const void* base, const FFDims& dm, int slices, int axis) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", (void**)&enc, cudaEnableDefault, &qr) != cudaSuccess || !enc)
      return false;
  }
  cuuint64_t dims[5] = {(cuuint64_t)CH, (cuuint64_t)dm.W, (cuuint64_t)dm.H, (cuuint64_t)dm.T, (cuuint64_t)slices};
  cuuint64_t strides[4] = {(cuuint64_t)CH * 2, (cuuint64_t)dm.W * CH * 2, (cuuint64_t)dm.H * dm.W * CH * 2,
                           (cuuint64_t)dm.N * CH * 2};
  cuuint32_t box[5] = {64, 1, 1, 1, 1};
  box[1 + (2 - axis)] = (cuuint32_t)(axis == 2 ? dm.W : (axis == 1 ? dm.H : dm.T));
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t launch_pass(ff_plan* p, const CUtensorMap& m0, const CUtensorMap& m1, const CUtensorMap& m2, DctTcParams& P,
                        cudaStream_t st) {
  const size_t img = (size_t)(P.n > 64 ? 2 : 1) * P.n * 128;
  const size_t stage = P.in_split ? 2 * TILE_BYTES : TILE_BYTES;
  const size_t fixed = 2 * img + sizeof(DctShared) + 1024;
  int nstage = (int)((220 * 1024 - fixed) / stage);
  if (nstage > MAX_STAGE) nstage = MAX_STAGE;
  P.nstage = nstage;
  const size_t smem = nstage * stage + fixed;
  cudaError_t e = cudaFuncSetAttribute(dct_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int lps = STAGE_ROWS / P.n;
  const int stages = (P.group * P.lines_per_th + lps - 1) / lps;
  const int grid = stages < p->sm_count ? stages : p->sm_count;
  dct_tc_kernel<<<grid, DCT_TC_THREADS, smem, st>>>(m0, m1, m2, P);
  p->launches += 1;
  return cudaGetLastError();
}

bool axis_ok(int n) { return n == 16 || n == 32 || n == 64 || n == 128; }

}  // namespace

// bf16, head_dim 128, power-of-two axis lengths 16..128, low box small enough for the fp32 side path.
bool ffk_dct_tc_supported(const FFDims& dm) {
  return !dm.fp32 && dm.d == CH && axis_ok(dm.T) && axis_ok(dm.H) && axis_ok(dm.W) && dm.L[2] <= 16;
}

// Scratch: two hi/lo pairs of bf16 grids and the fp32 side buffer for `group` tensor-heads.
size_t ffk_dct_tc_scratch_bytes(const FFDims& dm, int group) {
  const size_t grid = (size_t)group * dm.N * CH * 2;
  const size_t side = (size_t)group * dm.T * dm.H * dm.L[2] * CH * 4;
  return 4 * ((grid + 255) / 256 * 256) + (side + 255) / 256 * 256;
}

namespace {
struct Scratch { __nv_bfloat16 *a_hi, *a_lo, *b_hi, *b_lo; float* side; };
Scratch carve(ff_plan* p) {
  const size_t grid_bytes = ((size_t)p->dct_group * p->dm.N * CH * 2 + 255) / 256 * 256;
  char* base = (char*)p->buf.scratchA;
  Scratch s;
  s.a_hi = (__nv_bfloat16*)base; s.a_lo = (__nv_bfloat16*)(base + grid_bytes);
  s.b_hi = (__nv_bfloat16*)(base + 2 * grid_bytes); s.b_lo = (__nv_bfloat16*)(base + 3 * grid_bytes);
  s.side = (float*)(base + 4 * grid_bytes);
  return s;
}
}  // namespace

cudaError_t ffk_forward_transform_tc(ff_plan* p, const void* Q, const void* K, const void* V, bool want_energy,
                                     cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int G = p->dct_group;
  const Scratch sc = carve(p);
  float* side = sc.side;
  CUtensorMap mq, mk, mv, m1h, m1l, m2h, m2l;
  if (!encode_grid_map(&mq, Q, dm, dm.BH, 2) || !encode_grid_map(&mk, K, dm, dm.BH, 2) ||
      !encode_grid_map(&mv, V, dm, dm.BH, 2) || !encode_grid_map(&m1h, sc.a_hi, dm, G, 1) ||
      !encode_grid_map(&m1l, sc.a_lo, dm, G, 1) || !encode_grid_map(&m2h, sc.b_hi, dm, G, 0) ||
      !encode_grid_map(&m2l, sc.b_lo, dm, G, 0))
    return cudaErrorInvalidValue;
  const int total = 3 * dm.BH;
  DctTcParams P{};
  P.dm = dm; P.status = p->buf.status;
  P.spec_mid = (__nv_bfloat16*)p->buf.spec_mid; P.spec_high = (__nv_bfloat16*)p->buf.spec_high;
  P.energy = want_energy ? p->buf.energy : nullptr;
  for (int g0 = 0; g0 < total; g0 += G) {
    const int g = total - g0 < G ? total - g0 : G;
    P.group = g; P.group_start = g0;
    P.mode = MODE_FIRST; P.in_split = 0; P.axis = 2; P.n = dm.W; P.mat = p->basis[2]; P.lines_per_th = dm.T * dm.H;
    P.dst = sc.a_hi; P.dst_lo = sc.a_lo; P.side = side;
    cudaError_t e = launch_pass(p, mq, mk, mv, P, st);
    if (e != cudaSuccess) return e;
    P.mode = MODE_MIDDLE; P.in_split = 1; P.axis = 1; P.n = dm.H; P.mat = p->basis[1]; P.lines_per_th = dm.T * dm.W;
    P.dst = sc.b_hi; P.dst_lo = sc.b_lo;
    e = launch_pass(p, m1h, m1l, m1l, P, st);
    if (e != cudaSuccess) return e;
    P.mode = MODE_SPLIT; P.axis = 0; P.n = dm.T; P.mat = p->basis[0]; P.lines_per_th = dm.H * dm.W; P.dst = nullptr;
    e = launch_pass(p, m2h, m2l, m2l, P, st);
    if (e != cudaSuccess) return e;
    dim3 lgrid((unsigned)(dm.L[1] * dm.L[2]), (unsigned)g);
    low_band_kernel<<<lgrid, CH * LOW_TG, 0, st>>>(side, p->basis[0], p->basis[1], p->buf.spec_low, P.energy, dm, g0);
    p->launches += 1;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// Inverse transform of `g` recombined grids (hi/lo pair in the first scratch pair) into out[h0 .. h0+g).
cudaError_t ffk_inverse_transform_tc(ff_plan* p, int h0, int g, void* out, cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int G = p->dct_group;
  const Scratch sc = carve(p);
  CUtensorMap m_in, m_inl, mbh, mbl, mah, mal;
  if (!encode_grid_map(&m_in, sc.a_hi, dm, G, 0) || !encode_grid_map(&m_inl, sc.a_lo, dm, G, 0) ||
      !encode_grid_map(&mbh, sc.b_hi, dm, G, 1) ||
      !encode_grid_map(&mbl, sc.b_lo, dm, G, 1) || !encode_grid_map(&mah, sc.a_hi, dm, G, 2) ||
      !encode_grid_map(&mal, sc.a_lo, dm, G, 2))
    return cudaErrorInvalidValue;
  DctTcParams P{};
  P.dm = dm; P.status = p->buf.status; P.group = g; P.group_start = h0;
  P.mode = MODE_MIDDLE; P.in_split = 1; P.axis = 0; P.n = dm.T; P.mat = p->basis_t[0]; P.lines_per_th = dm.H * dm.W;
  P.dst = sc.b_hi; P.dst_lo = sc.b_lo;
  cudaError_t e = launch_pass(p, m_in, m_inl, m_inl, P, st);
  if (e != cudaSuccess) return e;
  P.in_split = 1; P.axis = 1; P.n = dm.H; P.mat = p->basis_t[1]; P.lines_per_th = dm.T * dm.W;
  P.dst = sc.a_hi; P.dst_lo = sc.a_lo;
  e = launch_pass(p, mbh, mbl, mbl, P, st);
  if (e != cudaSuccess) return e;
  P.mode = MODE_LAST; P.axis = 2; P.n = dm.W; P.mat = p->basis_t[2]; P.lines_per_th = dm.T * dm.H;
  P.dst = (__nv_bfloat16*)out; P.dst_lo = nullptr;
  return launch_pass(p, mah, mal, mal, P, st);
}
