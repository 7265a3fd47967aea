// Cross-band residual exchange + recombination on the tensor cores ("Cross-band residual
// exchange", "Reconstruction"), bf16 storage, head_dim 128 or 64 (template parameter XD), for the
// mid and high bands:
//     Y^[p] = Y[p] + softmax(Y[p] Z^T / sqrt(d)) Z,   Z = the 2m summary tokens of the other two bands
// written to the coefficient grid at the position of band rank p (a table built at plan creation).
//
// A CTA owns a contiguous run of (head, band, 128-rank tile) items, so the summary tokens of a head
// are re-staged only a few times per CTA.
// Two CTAs share an SM (256 tensor-memory columns each).  Inside a CTA the softmax warps work on
// tile n + 1 while the store warps finish tile n.  Per tile:
//   TMA     the 128 band tokens (operator output where the head's mask has the band, V~ otherwise)
//   MMA 1   S[128 x 3m] = Y Z^T against all 3m summaries of the head (own band masked in the softmax)
//   softmax one token per thread (row = TMEM lane); P written back to TMEM as bf16 hi + lo (normalised
//           for up to 32 keys, otherwise unnormalised with the row sum handed to the store warps)
//   MMA 2   D[128 x 128] = P Z  (A = P from tensor memory, B = the same Z image read MN-major)
//   store   Y + D in the three-byte form the inverse passes read (the value rounded to 24 bits: a grid of its
//           upper 16 bits and a grid of the next byte); a thread owns a token, the warp stages 32 channels of
//           its 32 tokens in shared memory and four lanes then write a token's 64 + 32 contiguous bytes
// Z and P are split into bf16 hi + lo parts (Y is exact bf16), so the logits and the update carry
// about 16 bits: the summary logits of a band with large low-frequency content reach O(100).
// The low band (fp32, a few hundred tokens) is handled by the generic kernel.
#include <cuda.h>

#include "ff_internal.h"
#include "ff_sm100.cuh"

using namespace sm100;

namespace {

constexpr int XT = 128;                 // tokens per tile
constexpr int XD_MAX = 128;             // largest head_dim; the shared-memory tiles are sized for it
constexpr int X_TILE_BYTES = XT * XD_MAX * 2;
constexpr int X_HALF = X_TILE_BYTES / 2;
constexpr int X_THREADS = 320;           // TMA warp, MMA warp, 4 softmax warps, 4 store warps

struct XParams {
  FFDims dm;
  const uint8_t* alloc;
  const float* summary;       // [BH][3][m][d]
  const int* pos_mid;         // [N_mid]  flat coefficient index of each band rank
  const int* pos_high;        // [N_high]
  __nv_bfloat16* grid_hi;     // [g][N][d]: upper 16 bits of the value rounded to 24 bits
  uint8_t* grid_lo;           // [g][N][d]: the next 8 bits (the three-byte form the inverse passes read)
  int h0, g;                  // heads [h0, h0+g)
  int nkeys;                  // 3m rounded up to a multiple of 16
  int ybufs;                  // token-tile buffers in shared memory (1 or 2)
  // With one buffer (two CTAs with two buffers each no longer fit an SM: more than 64 summary keys) the tile is
  // handed back to the producer as soon as the score MMAs have read it, and the store warps take the tokens for
  // the residual add from global memory instead (they were just loaded: L2 hits), so that the next tile's load
  // still overlaps this tile's softmax and stores.
  const __nv_bfloat16* src[4];   // y_mid, v~_mid, y_high, v~_high: bases of the buffers the four maps cover
  int* status;
};

#ifdef FF_X_PROF
__device__ unsigned long long g_x_prof[16];
#define XPROF_T0(v) const long long v = clock64()
#define XPROF_ADD(i, v) atomicAdd(&g_x_prof[i], (unsigned long long)(clock64() - (v)))
#else
#define XPROF_T0(v)
#define XPROF_ADD(i, v)
#endif

constexpr int X_STG_PITCH = 64;         // bytes per staged row piece (32 channels)

struct XShared {
  uint64_t y_full[2], y_empty[2], z_ready, s_full, p_full, d_full, d_empty;
  uint32_t tmem_base;
  int abort_flag;
  // per softmax warp: 32 rows x 64 bytes of hi and of lo (16-byte chunks XOR-swizzled with row / 2)
  alignas(16) uint8_t stage[4][2][32 * X_STG_PITCH];
  float inv[2][XT];          // (two-sweep variants) 1 / row sum of the tile, by tile parity
};

struct XItem { int bh, band, tile; };

__device__ __forceinline__ float ex2f_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ XItem x_decode(const FFDims& dm, int h0, int it, int tm, int th) {
  XItem x;
  const int per = tm + th;
  x.bh = h0 + it / per;
  const int rem = it % per;
  x.band = rem < tm ? 1 : 2;
  x.tile = rem < tm ? rem : rem - tm;
  return x;
}

// NK32 = 32-key chunks of the score row that are in use (3m <= 32 NK32).
// With two or three chunks the score row does not fit the registers two resident CTAs leave a
// thread: those variants sweep the scores twice (maximum, then exponentials chunk by chunk), write
// P unnormalised and let the store warps scale the update by 1 / row sum.  Their P_lo chunks sit in
// columns 96, 112 and 80, where no unread score can be overwritten.
template <int NK32, int XD>
__global__ void __launch_bounds__(X_THREADS, 2)
exchange_tc_kernel(const __grid_constant__ CUtensorMap map_y_mid, const __grid_constant__ CUtensorMap map_v_mid,
                   const __grid_constant__ CUtensorMap map_y_high, const __grid_constant__ CUtensorMap map_v_high,
                   const XParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sY = smem;                                    // ybufs x 32 KB
  uint8_t* sZhi = smem + P.ybufs * X_TILE_BYTES;         // [2 halves][nkeys rows][128 B]
  uint8_t* sZlo = sZhi + 2 * P.nkeys * 128;
  XShared& sh = *(XShared*)(sZlo + 2 * P.nkeys * 128);
  const FFDims& dm = P.dm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m = dm.m, nk = P.nkeys;
  const int tm_tiles = (int)((dm.Nmid + XT - 1) / XT), th_tiles = (int)((dm.Nhigh + XT - 1) / XT);
  const int total = P.g * (tm_tiles + th_tiles);
  const int chunk = (total + gridDim.x - 1) / gridDim.x;
  const int it0 = blockIdx.x * chunk;
  const int it1 = it0 + chunk < total ? it0 + chunk : total;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) { mbar_init(&sh.y_full[i], 1); mbar_init(&sh.y_empty[i], P.ybufs == 1 ? 1 : 128); }
    mbar_init(&sh.z_ready, 128); mbar_init(&sh.s_full, 1); mbar_init(&sh.p_full, 128);
    mbar_init(&sh.d_full, 1); mbar_init(&sh.d_empty, 128);
    sh.abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(&sh.tmem_base, 256); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;
  volatile int* abort_flag = &sh.abort_flag;
  // tensor-memory columns: S [0,96), overwritten by P_hi [0,48) and P_lo [48,96);  D [128,256)
  const int YB = P.ybufs;

  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      int n = 0;
      for (int it = it0; it < it1 && ok; ++it, ++n) {
        const XItem x = x_decode(dm, P.h0, it, tm_tiles, th_tiles);
        const bool exec = P.alloc[x.bh] & (1 << x.band);
        const CUtensorMap* map = x.band == 1 ? (exec ? &map_y_mid : &map_v_mid) : (exec ? &map_y_high : &map_v_high);
        const int slice = exec ? x.bh : 2 * dm.BH + x.bh;
        const int slot = n % YB;
        XPROF_T0(x0);
        if (n >= YB) ok = mbar_wait(&sh.y_empty[slot], ((n / YB) - 1) & 1, abort_flag);
        XPROF_ADD(0, x0);
        if (!ok) break;
        mbar_arrive_expect_tx(&sh.y_full[slot], XT * XD * 2);
        tma_load_3d(sY + slot * X_TILE_BYTES, map, &sh.y_full[slot], 0, x.tile * XT, slice);
        if (XD == 128) tma_load_3d(sY + slot * X_TILE_BYTES + X_HALF, map, &sh.y_full[slot], 64, x.tile * XT, slice);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc1 = idesc_bf16_f32(XT, nk, false, false);
      const uint32_t idesc2 = idesc_bf16_f32(XT, XD, false, true);
      const uint32_t zhi = smem_u32(sZhi), zlo = smem_u32(sZlo);
      const uint32_t zhalf = nk * 128;                    // bytes between the two 64-channel halves of a Z image
      bool ok = true;
      int n = 0, prev_bh = -1, zc = 0;
      for (int it = it0; it < it1 && ok; ++it, ++n) {
        const XItem x = x_decode(dm, P.h0, it, tm_tiles, th_tiles);
        if (x.bh != prev_bh) {                            // the softmax warps re-staged Z for this head
          XPROF_T0(x4);
          ok = mbar_wait(&sh.z_ready, zc & 1, abort_flag); ++zc; prev_bh = x.bh;
          XPROF_ADD(4, x4);
          if (!ok) break;
        }
        const int slot = n % YB;
        XPROF_T0(x1);
        ok = mbar_wait(&sh.y_full[slot], (n / YB) & 1, abort_flag);
        XPROF_ADD(1, x1);
        if (!ok) break;
        tc_fence_after();
        const uint32_t ybase = smem_u32(sY + slot * X_TILE_BYTES);
#pragma unroll
        for (int k = 0; k < XD / 16; ++k) {               // S = Y (Zhi + Zlo)^T, K = head_dim
          const uint64_t a = smem_desc_sw128(ybase + (k >> 2) * X_HALF + (k & 3) * 32, 16, 1024);
          const uint32_t zo = (k >> 2) * zhalf + (k & 3) * 32;
          umma_ss(tmem, a, smem_desc_sw128(zhi + zo, 16, 1024), idesc1, k > 0 ? 1u : 0u);
          umma_ss(tmem, a, smem_desc_sw128(zlo + zo, 16, 1024), idesc1, 1u);
        }
        umma_commit(&sh.s_full);
        if (YB == 1) umma_commit(&sh.y_empty[slot]);      // single buffer: free for the next load once the scores are done
        XPROF_T0(x2);
        ok = mbar_wait(&sh.p_full, n & 1, abort_flag);
        XPROF_ADD(2, x2);
        XPROF_T0(x3);
        if (ok && n >= 1) ok = mbar_wait(&sh.d_empty, (n - 1) & 1, abort_flag);
        XPROF_ADD(3, x3);
        if (!ok) break;
        tc_fence_after();
        for (int k = 0; k < nk / 16; ++k) {               // D = (Phi + Plo) (Zhi + Zlo) without lo*lo, K = keys
          const uint64_t bh_ = smem_desc_sw128(zhi + k * 2048, zhalf, 1024);
          umma_ts(tmem + 128, tmem + k * 8, bh_, idesc2, k > 0 ? 1u : 0u);
          umma_ts(tmem + 128, tmem + k * 8, smem_desc_sw128(zlo + k * 2048, zhalf, 1024), idesc2, 1u);
          const uint32_t plo = NK32 >= 2 ? (k < 2 ? 96u : (k < 4 ? 112u : 80u)) + (k & 1) * 8 : 48u + k * 8;
          umma_ts(tmem + 128, tmem + plo, bh_, idesc2, 1u);
        }
        umma_commit(&sh.d_full);
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ softmax warps
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const int tid = row;                                  // 0..127 among the softmax threads
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const float sl2 = rsqrtf((float)XD) * 1.4426950408889634f;
    // Keys a token attends to, as bit masks per 32-key chunk and band: the 3m summaries without the token's own
    // band's and without those of an empty mid band.
    uint32_t keys_mid[NK32], keys_high[NK32];
#pragma unroll
    for (int c3 = 0; c3 < NK32; ++c3) {
      uint32_t a = 0, b = 0;
      for (int i = 0; i < 32; ++i) {
        const int j = c3 * 32 + i;
        const bool live = j < 3 * m && !(dm.Nmid == 0 && j >= m && j < 2 * m);
        if (live && (j < m || j >= 2 * m)) a |= 1u << i;
        if (live && j < 2 * m) b |= 1u << i;
      }
      keys_mid[c3] = a; keys_high[c3] = b;
    }
    bool ok = true;
    int n = 0, prev_bh = -1;
    for (int it = it0; it < it1 && ok; ++it, ++n) {
      const XItem x = x_decode(dm, P.h0, it, tm_tiles, th_tiles);
      if (x.bh != prev_bh) {
        // Stage the head's 3m summaries as two bf16 images (hi, lo) in the operand layout: row = key,
        // 64 channels per 128-byte row, 16-byte chunks XOR-swizzled with the row.  Rows >= 3m are zero.
        // The MMAs of the previous tile, which read the old images, must have completed.
        prev_bh = x.bh;
        XPROF_T0(x8);
        if (n >= 1) {
          ok = __all_sync(0xffffffffu, mbar_wait(&sh.d_full, (n - 1) & 1, abort_flag));
          if (!ok) break;
        }
        if (tid == 0) XPROF_ADD(8, x8);
        XPROF_T0(x5);
        const float* S = P.summary + (size_t)x.bh * 3 * m * XD;
        for (int idx = tid; idx < nk * XD; idx += 128) {
          const int j = idx / XD, c = idx % XD;
          const float v = j < 3 * m ? S[j * XD + c] : 0.f;
          const __nv_bfloat16 hi = __float2bfloat16_rn(v);
          const __nv_bfloat16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
          const int half = c >> 6, ck = c & 63;
          const uint32_t off = half * (nk * 128) + j * 128 + ((((ck >> 3) ^ (j & 7)) << 4) | ((ck & 7) << 1));
          *(__nv_bfloat16*)(sZhi + off) = hi;
          *(__nv_bfloat16*)(sZlo + off) = lo;
        }
        fence_proxy_async();
        mbar_arrive(&sh.z_ready);
        if (tid == 0) XPROF_ADD(5, x5);
      }
      // ---- softmax over the 2m summaries of the other bands
      XPROF_T0(x6);
      ok = __all_sync(0xffffffffu, mbar_wait(&sh.s_full, n & 1, abort_flag));
      if (tid == 0) XPROF_ADD(6, x6);
      if (!ok) break;
      XPROF_T0(x7);
      tc_fence_after();
      uint32_t keys[NK32];
#pragma unroll
      for (int c3 = 0; c3 < NK32; ++c3) keys[c3] = x.band == 1 ? keys_mid[c3] : keys_high[c3];
      if (NK32 >= 2) {
        // first sweep: the row maximum
        float mx = -INFINITY;
#pragma unroll
        for (int c3 = 0; c3 < NK32; ++c3) {
          uint32_t r[32];
          tmem_ld32(tmem + lane_addr + c3 * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            if (keys[c3] & (1u << i)) mx = fmaxf(mx, __uint_as_float(r[i]));
          }
        }
        const float mb = mx * sl2;
        // second sweep: exponentials and their sum, P (unnormalised, bf16 hi + lo) chunk by chunk
        float den0 = 0.f, den1 = 0.f;
#pragma unroll
        for (int c3 = 0; c3 < NK32; ++c3) {
          uint32_t r[32];
          tmem_ld32(tmem + lane_addr + c3 * 32, r);
          tmem_wait_ld();
          uint32_t ph[16], pl[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            float p0 = 0.f, p1 = 0.f;
            if (keys[c3] & (1u << (2 * i))) p0 = ex2f_approx(fmaf(__uint_as_float(r[2 * i]), sl2, -mb));
            if (keys[c3] & (2u << (2 * i))) p1 = ex2f_approx(fmaf(__uint_as_float(r[2 * i + 1]), sl2, -mb));
            den0 += p0; den1 += p1;
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
            ph[i] = *(const uint32_t*)&h2;
            const __nv_bfloat162 l2 = __floats2bfloat162_rn(p0 - __uint_as_float(ph[i] << 16), p1 - __uint_as_float(ph[i] & 0xffff0000u));
            pl[i] = *(const uint32_t*)&l2;
          }
          tmem_st16(tmem + lane_addr + c3 * 16, ph);                              // over scores already read
          tmem_st16(tmem + lane_addr + (c3 == 0 ? 96 : (c3 == 1 ? 112 : 80)), pl);
        }
        sh.inv[n & 1][row] = 1.f / (den0 + den1);
      } else {
      // all scores of the row into registers (they are overwritten by P below)
        uint32_t sc[NK32 * 32];
#pragma unroll
        for (int c3 = 0; c3 < NK32; ++c3) {
          uint32_t r[32];
          tmem_ld32(tmem + lane_addr + c3 * 32, r);
#pragma unroll
          for (int i = 0; i < 32; ++i) sc[c3 * 32 + i] = r[i];
        }
        tmem_wait_ld();
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int j = 0; j < NK32 * 32; ++j)
          if (keys[j >> 5] & (1u << (j & 31))) mx4[j & 3] = fmaxf(mx4[j & 3], __uint_as_float(sc[j]));
        const float mb = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sl2;
        float den4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int j = 0; j < NK32 * 32; ++j) {
          float pv = 0.f;
          if (keys[j >> 5] & (1u << (j & 31))) pv = ex2f_approx(fmaf(__uint_as_float(sc[j]), sl2, -mb));
          den4[j & 3] += pv;
          sc[j] = __float_as_uint(pv);
        }
        const float inv = 1.f / ((den4[0] + den4[1]) + (den4[2] + den4[3]));
#pragma unroll
        for (int c3 = 0; c3 < NK32; ++c3) {
          if (c3 * 32 < nk) {
            uint32_t ph[16], pl[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float p0 = __uint_as_float(sc[c3 * 32 + 2 * i]) * inv, p1 = __uint_as_float(sc[c3 * 32 + 2 * i + 1]) * inv;
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
              ph[i] = *(const uint32_t*)&h2;
              const __nv_bfloat162 l2 = __floats2bfloat162_rn(p0 - __uint_as_float(ph[i] << 16), p1 - __uint_as_float(ph[i] & 0xffff0000u));
              pl[i] = *(const uint32_t*)&l2;
            }
            tmem_st16(tmem + lane_addr + c3 * 16, ph);
            tmem_st16(tmem + lane_addr + 48 + c3 * 16, pl);
          }
        }
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&sh.p_full);
      if (tid == 0) XPROF_ADD(7, x7);
    }
  } else {
    // ------------------------------------------------------------------ store warps
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    bool ok = true;
    int n = 0;
    for (int it = it0; it < it1 && ok; ++it, ++n) {
      const XItem x = x_decode(dm, P.h0, it, tm_tiles, th_tiles);
      const int slot = n % YB;
      const long long n_band = x.band == 1 ? dm.Nmid : dm.Nhigh;
      const long long p = (long long)x.tile * XT + row;
      // ---- residual add and store (where the rows go does not depend on the data: looked up before the wait)
      const bool valid = p < n_band;
      XPROF_T0(x14);
      int f = valid ? (x.band == 1 ? P.pos_mid[p] : P.pos_high[p]) : -1;
      if (valid && !FF_DBG_OK(f >= 0 && f < dm.N && x.bh >= P.h0 && x.bh < P.h0 + P.g, P.status, 3)) f = -1;   // (debug build)
      // lane L stores for rows 8 i + L/4 of its warp: fetch those rows' grid positions
      int fpos[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) fpos[i] = __shfl_sync(0xffffffffu, f, 8 * i + (lane >> 2));
      const size_t obase = (size_t)(x.bh - P.h0) * dm.N * XD;
      const uint8_t* yrow = sY + slot * X_TILE_BYTES + row * 128;
      // (single buffer) this token's row in global memory; rows past the band end are never stored
      const bool exec_g = P.alloc[x.bh] & (1 << x.band);
      const __nv_bfloat16* grow = P.src[(x.band == 1 ? 0 : 2) + (exec_g ? 0 : 1)] +
                                  ((size_t)(exec_g ? x.bh : 2 * dm.BH + x.bh) * n_band + (valid ? p : 0)) * XD;
      uint8_t* st_hi = sh.stage[quarter][0];
      uint8_t* st_lo = sh.stage[quarter][1];
      if (row == 0) XPROF_ADD(14, x14);
      XPROF_T0(x9);
      ok = __all_sync(0xffffffffu, mbar_wait(&sh.d_full, n & 1, abort_flag));
      if (row == 0) XPROF_ADD(9, x9);
      if (!ok) break;
      XPROF_T0(x10);
      tc_fence_after();
      const float dscale = NK32 >= 2 ? sh.inv[n & 1][row] : 1.f;    // (two-sweep variants: P was left unnormalised)
#pragma unroll
      for (int q = 0; q < XD / 32; ++q) {
        uint32_t r[32];
        XPROF_T0(x11);
        tmem_ld32(tmem + lane_addr + 128 + q * 32, r);
        tmem_wait_ld();
        if (row == 0) XPROF_ADD(11, x11);
        XPROF_T0(x12);
#pragma unroll
        for (int v4 = 0; v4 < 4; ++v4) {
          // channels 32q + 8v4 .. +7 of this token: one 16-byte chunk of the swizzled Y tile
          const int cch = q * 4 + v4;                    // 16-byte chunk index along the row, 0..15
          const uint4 yv = YB == 1 ? __ldg((const uint4*)(grow + cch * 8))
                                   : *(const uint4*)(yrow + (cch >> 3) * X_HALF + (((cch & 7) ^ (row & 7)) << 4));
          const uint32_t yw[4] = {yv.x, yv.y, yv.z, yv.w};
          // three-byte form: the value rounded to 24 bits; hi = its upper 16 bits, lo = the next byte
          uint32_t hi[4], u[8];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            u[2 * i] = __float_as_uint(fmaf(__uint_as_float(r[v4 * 8 + 2 * i]), dscale, __uint_as_float(yw[i] << 16))) + 0x80u;
            u[2 * i + 1] = __float_as_uint(fmaf(__uint_as_float(r[v4 * 8 + 2 * i + 1]), dscale, __uint_as_float(yw[i] & 0xffff0000u))) + 0x80u;
            hi[i] = __byte_perm(u[2 * i], u[2 * i + 1], 0x7632);
          }
          const uint32_t lo0 = __byte_perm(__byte_perm(u[0], u[1], 0x0051), __byte_perm(u[2], u[3], 0x0051), 0x5410);
          const uint32_t lo1 = __byte_perm(__byte_perm(u[4], u[5], 0x0051), __byte_perm(u[6], u[7], 0x0051), 0x5410);
          *(uint4*)(st_hi + lane * X_STG_PITCH + ((v4 ^ ((lane >> 1) & 3)) << 4)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          // (lo: 32 bytes per row, 8-byte pieces XOR-swizzled with row / 4)
          *(uint2*)(st_lo + lane * 32 + ((v4 ^ ((lane >> 2) & 3)) << 3)) = make_uint2(lo0, lo1);
        }
        __syncwarp();
        if (row == 0) XPROF_ADD(12, x12);
        XPROF_T0(x13);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int rr = 8 * i + (lane >> 2), piece = lane & 3;      // row of the warp, 16-byte piece of its 64 bytes
          if (fpos[i] >= 0) {
            const size_t o = obase + (size_t)fpos[i] * XD + q * 32 + piece * 8;
            const int so = rr * X_STG_PITCH + ((piece ^ ((rr >> 1) & 3)) << 4);
            *(uint4*)(P.grid_hi + o) = *(const uint4*)(st_hi + so);
            *(uint2*)(P.grid_lo + o) = *(const uint2*)(st_lo + rr * 32 + ((piece ^ ((rr >> 2) & 3)) << 3));
          }
        }
        __syncwarp();
        if (row == 0) XPROF_ADD(13, x13);
      }
      tc_fence_before();
      mbar_arrive(&sh.d_empty);
      if (YB > 1) mbar_arrive(&sh.y_empty[slot]);
      if (row == 0) XPROF_ADD(10, x10);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (sh.abort_flag) {
    if (threadIdx.x == 0) atomicExch(P.status, FF_ERR_TIMEOUT | 0x300);   // low byte: status, next byte: which kernel
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool encode_rows_map(CUtensorMap* map, void* base, long long rows, int slices, int d) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", (void**)&enc, cudaEnableDefault, &qr) != cudaSuccess || !enc)
      return false;
  }
  cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)rows, (cuuint64_t)slices};
  cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)rows * d * 2};
  cuuint32_t box[3] = {64, XT, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

#ifdef FF_X_PROF
extern "C" void ff_debug_x_prof(unsigned long long* out16, int reset) {
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(out16, g_x_prof, sizeof(unsigned long long) * 16);
  if (reset) { unsigned long long z[16] = {}; cudaMemcpyToSymbol(g_x_prof, z, sizeof(z)); }
}
#endif

bool ffk_exchange_tc_supported(const FFDims& dm) {
  return !dm.fp32 && (dm.d == 128 || dm.d == 64) && dm.m >= 1 && dm.m <= 32 && dm.N < (1LL << 31);
}

// Rank -> flat coefficient index tables of the mid and high bands (plan-owned device memory).
bool ffk_exchange_tc_build_tables(ff_plan* p) {
  const FFDims& dm = p->dm;
  int* host = (int*)malloc((size_t)(dm.Nmid + dm.Nhigh) * sizeof(int));
  if (!host) return false;
  for (int kt = 0; kt < dm.T; ++kt)
    for (int kh = 0; kh < dm.H; ++kh)
      for (int kw = 0; kw < dm.W; ++kw) {
        long long rank;
        const int band = ff_band_rank_of(dm, kt, kh, kw, &rank);
        const int f = (kt * dm.H + kh) * dm.W + kw;
        if (band == 1) host[rank] = f;
        else if (band == 2) host[dm.Nmid + rank] = f;
      }
  bool ok = cudaMalloc((void**)&p->pos_table, (size_t)(dm.Nmid + dm.Nhigh) * sizeof(int)) == cudaSuccess &&
            cudaMemcpy(p->pos_table, host, (size_t)(dm.Nmid + dm.Nhigh) * sizeof(int), cudaMemcpyHostToDevice) == cudaSuccess;
  free(host);
  return ok;
}

bool ffk_exchange_tc_prepare(ff_plan* p) {
  const FFDims& dm = p->dm;
  // (an empty mid band has no tiles; its maps are encoded over one row of the high band's buffers and never used)
  const long long nm = dm.Nmid > 0 ? dm.Nmid : 1;
  return encode_rows_map((CUtensorMap*)p->tmap_x[0], dm.Nmid > 0 ? p->buf.y_mid : p->buf.y_high, nm, dm.BH, dm.d) &&
         encode_rows_map((CUtensorMap*)p->tmap_x[1], dm.Nmid > 0 ? p->buf.spec_mid : p->buf.spec_high, nm, 3 * dm.BH, dm.d) &&
         encode_rows_map((CUtensorMap*)p->tmap_x[2], p->buf.y_high, dm.Nhigh, dm.BH, dm.d) &&
         encode_rows_map((CUtensorMap*)p->tmap_x[3], p->buf.spec_high, dm.Nhigh, 3 * dm.BH, dm.d);
}

// Exchange + recombination of the mid and high bands of heads [h0, h0+g) into the hi/lo grids.
cudaError_t ffk_exchange_tc(ff_plan* p, int h0, int g, void* grid_hi, void* grid_lo, cudaStream_t st) {
  const FFDims& dm = p->dm;
  XParams P;
  P.dm = dm; P.alloc = p->buf.alloc; P.summary = p->buf.summary;
  P.pos_mid = p->pos_table; P.pos_high = p->pos_table + dm.Nmid;
  P.grid_hi = (__nv_bfloat16*)grid_hi; P.grid_lo = (uint8_t*)grid_lo;
  P.h0 = h0; P.g = g; P.nkeys = (3 * dm.m + 15) / 16 * 16; P.status = p->buf.status;
  P.src[0] = (const __nv_bfloat16*)p->buf.y_mid; P.src[1] = (const __nv_bfloat16*)p->buf.spec_mid;
  P.src[2] = (const __nv_bfloat16*)p->buf.y_high; P.src[3] = (const __nv_bfloat16*)p->buf.spec_high;
  // Two CTAs per SM; the token tile is double-buffered if both still fit in shared memory
  const int per_sm = 2;
  P.ybufs = (2 * X_TILE_BYTES + 4 * P.nkeys * 128 + sizeof(XShared) + 2048) * per_sm <= 227 * 1024 ? 2 : 1;
  const size_t smem = P.ybufs * X_TILE_BYTES + 4 * P.nkeys * 128 + sizeof(XShared) + 1024;
  const long long tiles = (long long)g * ((dm.Nmid + XT - 1) / XT + (dm.Nhigh + XT - 1) / XT);
  const int grid = tiles < per_sm * p->sm_count ? (int)tiles : per_sm * p->sm_count;
  const CUtensorMap& m0 = *(const CUtensorMap*)p->tmap_x[0];
  const CUtensorMap& m1 = *(const CUtensorMap*)p->tmap_x[1];
  const CUtensorMap& m2 = *(const CUtensorMap*)p->tmap_x[2];
  const CUtensorMap& m3 = *(const CUtensorMap*)p->tmap_x[3];
  cudaError_t e = cudaSuccess;
#define FF_XCH(NK, D)                                                                                              \
  do {                                                                                                             \
    e = cudaFuncSetAttribute(exchange_tc_kernel<NK, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);   \
    if (e == cudaSuccess) exchange_tc_kernel<NK, D><<<grid, X_THREADS, smem, st>>>(m0, m1, m2, m3, P);             \
  } while (0)
  if (dm.d == 128) {
    if (P.nkeys <= 32) FF_XCH(1, 128); else if (P.nkeys <= 64) FF_XCH(2, 128); else FF_XCH(3, 128);
  } else {
    if (P.nkeys <= 32) FF_XCH(1, 64); else if (P.nkeys <= 64) FF_XCH(2, 64); else FF_XCH(3, 64);
  }
#undef FF_XCH
  if (e != cudaSuccess) return e;
  p->launches += 1;
  return cudaGetLastError();
}
