// The w- and h-axis passes of the separable transform fused into one persistent launch, for grids
// with H == W ("Separable spectral decomposition", "Reconstruction").  Both passes act inside one
// t-slab (all h, all w of one t), so the intermediate between them is written to a small ring of slab
// buffers and read back while it is still in L2, instead of travelling through HBM:
//   forward   Q/K/V --w pass--> ring (hi/lo, + the fp32 rows k_w < L_w) --h pass--> hi/lo grid
//   inverse   hi/lo grid --h pass--> ring (hi/lo) --w pass--> the caller's out tensor
// The t-axis pass stays a separate launch (ff_dct_tc.cu): it needs every slab of a tensor-head.
//
// Work is one static queue of 128-position tiles: group k holds the first-pass tiles of slab k and
// the second-pass tiles of slab k - lag; CTA i takes entries i, i + grid, ...  A second-pass tile
// waits (bounded) until the slab's first-pass tiles have all been stored, a first-pass tile until the
// ring slot it overwrites has been consumed; both conditions refer to earlier queue entries only,
// so the earliest unfinished entry can always proceed.  Per-slab counters in global memory carry
// the dependencies (one release per epilogue warp, acquire + cross-proxy fence before the TMA load).
// An epilogue warp sends its rows out with tensor stores and releases a tile's counter only when
// the stores have completed, which it checks after its next tile (so that the completion latency is
// off the critical path); the launcher only fuses when no tile can depend on a release that is still
// deferred in this way (lag * 2 * tiles-per-slab > grid + tiles-per-slab, lag not clamped).
// Ring traffic carries an evict-last L2 policy, the streamed input and output evict-first.
//
// Tile math, precision (hi/lo split of matrix and intermediates) and the warp roles are those of
// dct_tc_kernel: A = I kron Mat image (K-major), B = the TMA tile in place (MN-major), D in tensor
// memory with one output position per lane.  Both passes use lines that follow one another inside
// a tile (the h pass fetches its 128/n lines with one TMA box each), so one matrix image serves both.
#include <cuda.h>

#include "ff_internal.h"
#include "ff_sm100.cuh"

using namespace sm100;

namespace {

constexpr int CH = 128;
constexpr int TILE_ROWS = 128;
constexpr int TILE_BYTES = TILE_ROWS * CH * 2;     // 32 KB
constexpr int HALF_BYTES = TILE_BYTES / 2;
constexpr int STAGE_BYTES = 2 * TILE_BYTES;        // hi + lo
constexpr int NSTAGE = 2;
constexpr int NACC = 4;
constexpr int WH_THREADS = 320;        // TMA warp, MMA warp, 8 epilogue warps
constexpr int STG_PITCH = 64;                       // bytes per staged row piece (64-byte swizzle of the store maps)

struct WhParams {
  FFDims dm;
  const uint8_t* image;        // hi then lo image of I kron Mat, 32 KB each
  int n;                       // H == W
  int forward;                 // 1: w pass then h pass;  0: h pass then w pass
  int group, group_start;      // tensor-heads of this launch (forward: tensor*BH + bh; inverse: bh)
  int ring, lag;               // ring slots, and how many slabs the second pass trails the first
  int* cnt_a;                  // [slabs] first-pass epilogue warps done
  int* cnt_b;                  // [slabs] second-pass epilogue warps done
  float* side;                 // forward: [group][T][H][L_w][128] fp32
  int* status;
};

struct WhShared {
  uint64_t full[NSTAGE], empty[NSTAGE], acc_full[NACC], acc_empty[NACC], img_full;
  uint32_t tmem_base;
  int abort_flag;
  alignas(1024) uint8_t stage[8][2][32 * STG_PITCH];
};

struct WhTile {
  int second;      // 0: first pass, 1: second pass
  int slab;        // gi * T + t
  int u;           // tile inside the slab
};

// Queue entry -> tile.  tps = tiles per slab and pass, S = slabs, D = lag (D <= S).
__device__ __forceinline__ WhTile wh_decode(int idx, int tps, int S, int D) {
  WhTile x;
  const int head = D * tps, mid = (S - D) * 2 * tps;
  if (idx < head) { x.second = 0; x.slab = idx / tps; x.u = idx % tps; }
  else if (idx < head + mid) {
    const int i2 = idx - head, k = D + i2 / (2 * tps), r = i2 % (2 * tps);
    if (r < tps) { x.second = 0; x.slab = k; x.u = r; } else { x.second = 1; x.slab = k - D; x.u = r - tps; }
  } else {
    const int i3 = idx - head - mid;
    x.second = 1; x.slab = S - D + i3 / tps; x.u = i3 % tps;
  }
  return x;
}

__device__ __forceinline__ void tma_load_5d(void* smem_dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2,
                                            int c3, int c4, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6, %7}], [%2], %8;"
      ::"r"(smem_u32(smem_dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "l"(policy)
      : "memory");
}

__device__ __forceinline__ void tma_store_5d(const void* smem_src, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                             int c4, uint64_t policy) {
  asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3, %4, %5, %6}], [%1], %7;"
               ::"l"((uint64_t)map), "r"(smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "l"(policy)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait2() { asm volatile("cp.async.bulk.wait_group 2;" ::: "memory"); }

__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"((uint64_t)gsrc), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// Bounded wait until *cnt >= target (acquire), then order the TMA reads that follow after the
// generic-proxy stores the counter stands for.
__device__ __forceinline__ bool wait_counter(const int* cnt, int target, volatile int* abort_flag) {
  const long long t0 = clock64();
  while (true) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(cnt) : "memory");
    if (v >= target) break;
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitLimitCycles) { *abort_flag = 1; return false; }
  }
  asm volatile("fence.proxy.async.global;" ::: "memory");
  return true;
}

// The same with the counter already sampled (a relaxed load issued one tile earlier, so that its
// latency overlaps the previous tile's copies): if the sample suffices, an acquire fence orders the
// reads that follow; otherwise poll.
__device__ __forceinline__ bool wait_counter_sampled(const int* cnt, int sample, int target, volatile int* abort_flag) {
  if (sample < target) return wait_counter(cnt, target, abort_flag);
  asm volatile("fence.acquire.gpu;" ::: "memory");
  asm volatile("fence.proxy.async.global;" ::: "memory");
  return true;
}

__device__ __forceinline__ int load_relaxed(const int* p) {
  int v;
  asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// m0..m2: first-pass input (forward: Q, K, V; inverse: hi grid, lo grid, unused).
// m3, m4: the ring (hi, lo) with the box of the second pass.
// s_rh, s_rl: store maps of the ring (box of an epilogue warp of the first pass); s_oh, s_ol: store
// maps of the result (box of an epilogue warp of the second pass; the inverse has no lo result).
__global__ void __launch_bounds__(WH_THREADS, 1)
dct_wh_kernel(const __grid_constant__ CUtensorMap m0, const __grid_constant__ CUtensorMap m1,
              const __grid_constant__ CUtensorMap m2, const __grid_constant__ CUtensorMap m3,
              const __grid_constant__ CUtensorMap m4, const __grid_constant__ CUtensorMap s_rh,
              const __grid_constant__ CUtensorMap s_rl, const __grid_constant__ CUtensorMap s_oh,
              const __grid_constant__ CUtensorMap s_ol, const WhParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sData = smem;                                  // NSTAGE x 64 KB
  uint8_t* sHi = smem + NSTAGE * STAGE_BYTES;
  uint8_t* sLo = sHi + TILE_BYTES;
  WhShared& sh = *(WhShared*)(sLo + TILE_BYTES);
  const FFDims& dm = P.dm;
  const int n = P.n, kf = TILE_ROWS / n, ln = 31 - __clz(n);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tps = (n * n) / TILE_ROWS;                    // tiles per slab and pass
  const int S = P.group * dm.T, D = P.lag;
  const int total = 2 * S * tps;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NSTAGE; ++i) { mbar_init(&sh.full[i], 1); mbar_init(&sh.empty[i], 1); }
    for (int i = 0; i < NACC; ++i) { mbar_init(&sh.acc_full[i], 1); mbar_init(&sh.acc_empty[i], 256); }
    mbar_init(&sh.img_full, 1);
    sh.abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = sh.tmem_base;
  volatile int* abort_flag = &sh.abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      mbar_arrive_expect_tx(&sh.img_full, 2 * TILE_BYTES);
      bulk_load(sHi, P.image, TILE_BYTES, &sh.img_full);
      bulk_load(sLo, P.image + TILE_BYTES, TILE_BYTES, &sh.img_full);
      const uint64_t pol_ring = policy_evict_last(), pol_stream = policy_evict_first();
      unsigned it = 0;
      bool ok = true;
      // the counter a tile depends on: the slab's first pass is stored / the ring slot has been consumed
      auto counter_of = [&](const WhTile& y) -> const int* {
        return y.second ? P.cnt_a + y.slab : (y.slab >= P.ring ? P.cnt_b + y.slab - P.ring : nullptr);
      };
      const int* cnt_next = blockIdx.x < total ? counter_of(wh_decode(blockIdx.x, tps, S, D)) : nullptr;
      int sample_next = cnt_next ? load_relaxed(cnt_next) : 0;
      for (int idx = blockIdx.x; idx < total && ok; idx += gridDim.x, ++it) {
        const WhTile x = wh_decode(idx, tps, S, D);
        const int gi = x.slab / dm.T, t = x.slab % dm.T, slot = x.slab % P.ring;
        const bool along_w = (x.second == 0) == (P.forward != 0);
        const bool split = x.second || !P.forward;
        const uint64_t pol = x.second ? pol_ring : pol_stream;
        const int* cnt = cnt_next;
        const int sample = sample_next;
        // sample the next tile's counter now; it is looked at one iteration later
        cnt_next = idx + (int)gridDim.x < total ? counter_of(wh_decode(idx + gridDim.x, tps, S, D)) : nullptr;
        sample_next = cnt_next ? load_relaxed(cnt_next) : 0;
        if (cnt) ok = wait_counter_sampled(cnt, sample, 8 * tps, abort_flag);
        if (!ok) break;
        const int st = it % NSTAGE;
        if (it >= NSTAGE) ok = mbar_wait(&sh.empty[st], ((it / NSTAGE) - 1) & 1, abort_flag);
        if (!ok) break;
        uint8_t* dst = sData + st * STAGE_BYTES;
        const CUtensorMap* mhi; const CUtensorMap* mlo = nullptr;
        int tc, slice;
        if (x.second) { mhi = &m3; mlo = &m4; tc = slot; slice = 0; }
        else if (P.forward) {
          const int th = P.group_start + gi, tensor = th / dm.BH;
          mhi = tensor == 0 ? &m0 : (tensor == 1 ? &m1 : &m2); tc = t; slice = th % dm.BH;
        } else { mhi = &m0; mlo = &m1; tc = t; slice = gi; }
        mbar_arrive_expect_tx(&sh.full[st], split ? STAGE_BYTES : TILE_BYTES);
        if (along_w) {                                    // one box: kf whole lines along w
          const int h0 = x.u * kf;
          tma_load_5d(dst, mhi, &sh.full[st], 0, 0, h0, tc, slice, pol);
          tma_load_5d(dst + HALF_BYTES, mhi, &sh.full[st], 64, 0, h0, tc, slice, pol);
          if (split) {
            tma_load_5d(dst + TILE_BYTES, mlo, &sh.full[st], 0, 0, h0, tc, slice, pol);
            tma_load_5d(dst + TILE_BYTES + HALF_BYTES, mlo, &sh.full[st], 64, 0, h0, tc, slice, pol);
          }
        } else {                                          // kf boxes: one line along h each
          const int w0 = x.u * kf;
          for (int l = 0; l < kf; ++l) {
            const int o = l * n * 128;
            tma_load_5d(dst + o, mhi, &sh.full[st], 0, w0 + l, 0, tc, slice, pol);
            tma_load_5d(dst + HALF_BYTES + o, mhi, &sh.full[st], 64, w0 + l, 0, tc, slice, pol);
            if (split) {
              tma_load_5d(dst + TILE_BYTES + o, mlo, &sh.full[st], 0, w0 + l, 0, tc, slice, pol);
              tma_load_5d(dst + TILE_BYTES + HALF_BYTES + o, mlo, &sh.full[st], 64, w0 + l, 0, tc, slice, pol);
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(TILE_ROWS, CH, /*a_mn_major=*/false, /*b_mn_major=*/true);
      const uint32_t hi_base = smem_u32(sHi), lo_base = smem_u32(sLo);
      unsigned it = 0;
      bool ok = mbar_wait(&sh.img_full, 0, abort_flag);
      for (int idx = blockIdx.x; idx < total && ok; idx += gridDim.x, ++it) {
        const WhTile x = wh_decode(idx, tps, S, D);
        const bool split = x.second || !P.forward;
        const int st = it % NSTAGE, ab = it % NACC;
        ok = mbar_wait(&sh.full[st], (it / NSTAGE) & 1, abort_flag);
        if (ok && it >= NACC) ok = mbar_wait(&sh.acc_empty[ab], ((it / NACC) - 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t dbase = smem_u32(sData + st * STAGE_BYTES);
        const uint32_t d_tm = tm + ab * 128;
#pragma unroll
        for (int ks = 0; ks < TILE_ROWS / 16; ++ks) {
          const uint32_t aoff = (ks >> 2) * HALF_BYTES + (ks & 3) * 32;
          const uint64_t ahi = smem_desc_sw128(hi_base + aoff, 16, 1024);
          const uint64_t xhi = smem_desc_sw128(dbase + ks * 2048, HALF_BYTES, 1024);
          umma_ss(d_tm, ahi, xhi, idesc, ks > 0 ? 1u : 0u);
          umma_ss(d_tm, smem_desc_sw128(lo_base + aoff, 16, 1024), xhi, idesc, 1u);
          if (split) umma_ss(d_tm, ahi, smem_desc_sw128(dbase + TILE_BYTES + ks * 2048, HALF_BYTES, 1024), idesc, 1u);
        }
        umma_commit(&sh.empty[st]);
        umma_commit(&sh.acc_full[ab]);
      }
    }
  } else {
    const int quarter = warp & 3;
    const int j = quarter * 32 + lane;                    // output position of this thread inside a tile
    const int a = j & (n - 1), l = j >> ln;               // output index along the axis, line of the tile
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const int ew = warp - 2;                              // epilogue warp 0..7: warps 0-3 take channels 0..63, 4-7 channels 64..127
    const int q_lo = (ew >> 2) * 2;
    const uint64_t pol_ring = policy_evict_last(), pol_stream = policy_evict_first();
    int* pending = nullptr;                               // counter of the tile whose stores are still in flight
    unsigned it = 0;
    bool ok = true;
    for (int idx = blockIdx.x; idx < total && ok; idx += gridDim.x, ++it) {
      const WhTile x = wh_decode(idx, tps, S, D);
      const int gi = x.slab / dm.T, t = x.slab % dm.T, slot = x.slab % P.ring;
      const bool along_w = (x.second == 0) == (P.forward != 0);
      const int ab = it % NACC;
      ok = __all_sync(0xffffffffu, mbar_wait(&sh.acc_full[ab], (it / NACC) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      // grid position (h, w) of this thread's output row (for the fp32 side rows) and of the warp's
      // first row: the warp's 32 rows are 32 consecutive positions along the pass axis
      const int h = along_w ? x.u * kf + l : a;
      const int j0 = quarter * 32, a0 = j0 & (n - 1), l0 = j0 >> ln;
      const int bh0 = along_w ? x.u * kf + l0 : a0, bw0 = along_w ? a0 : x.u * kf + l0;
      float* row_f32 = nullptr;
      if (!x.second && P.forward && P.side && a < dm.L[2]) row_f32 = P.side + ((((size_t)gi * dm.T + t) * dm.H + h) * dm.L[2] + a) * CH;
      const CUtensorMap* mo_hi; const CUtensorMap* mo_lo;
      int c3, c4;
      uint64_t pol;
      bool want_lo = true;
      if (!x.second) { mo_hi = &s_rh; mo_lo = &s_rl; c3 = slot; c4 = 0; pol = pol_ring; }
      else if (P.forward) { mo_hi = &s_oh; mo_lo = &s_ol; c3 = t; c4 = gi; pol = pol_stream; }
      else { mo_hi = &s_oh; mo_lo = &s_ol; c3 = t; c4 = P.group_start + gi; pol = pol_stream; want_lo = false; }
#pragma unroll
      for (int q = q_lo; q < q_lo + 2; ++q) {
        uint32_t r[32];
        tmem_ld32(tm + lane_addr + ab * 128 + q * 32, r);
        tmem_wait_ld();
        if (row_f32) {
#pragma unroll
          for (int i = 0; i < 8; ++i)
            *(uint4*)(row_f32 + q * 32 + i * 4) = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
        }
        uint32_t hi[16], lo[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const __nv_bfloat162 hp = __floats2bfloat162_rn(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
          hi[i] = *(const uint32_t*)&hp;
        }
        if (want_lo) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const __nv_bfloat162 lp = __floats2bfloat162_rn(__uint_as_float(r[2 * i]) - __uint_as_float(hi[i] << 16),
                                                           __uint_as_float(r[2 * i + 1]) - __uint_as_float(hi[i] & 0xffff0000u));
            lo[i] = *(const uint32_t*)&lp;
          }
        }
        uint8_t* st_hi = sh.stage[ew][0];
        uint8_t* st_lo = sh.stage[ew][1];
        // the previous store of this warp must have read the staging area
        if (lane == 0) bulk_wait_read0();
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          *(uint4*)(st_hi + lane * STG_PITCH + ((i ^ ((lane >> 1) & 3)) << 4)) = make_uint4(hi[4 * i], hi[4 * i + 1], hi[4 * i + 2], hi[4 * i + 3]);
          if (want_lo)
            *(uint4*)(st_lo + lane * STG_PITCH + ((i ^ ((lane >> 1) & 3)) << 4)) = make_uint4(lo[4 * i], lo[4 * i + 1], lo[4 * i + 2], lo[4 * i + 3]);
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          tma_store_5d(st_hi, mo_hi, q * 32, bw0, bh0, c3, c4, pol);
          if (want_lo) tma_store_5d(st_lo, mo_lo, q * 32, bw0, bh0, c3, c4, pol);
          bulk_commit();
        }
      }
      tc_fence_before();
      mbar_arrive(&sh.acc_empty[ab]);
      // publish the PREVIOUS tile of this warp: its two store groups are complete once at most this
      // tile's two are pending (release after completion; the reader acquires the counter and fences
      // towards the async proxy before its TMA load)
      if (lane == 0) {
        if (pending) {
          bulk_wait2();
          asm volatile("fence.proxy.async.global;" ::: "memory");
          asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(pending) : "memory");
        }
        pending = (x.second ? P.cnt_b : P.cnt_a) + x.slab;
      }
    }
    if (lane == 0) {
      bulk_wait0();
      if (pending) {
        asm volatile("fence.proxy.async.global;" ::: "memory");
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(pending) : "memory");
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (sh.abort_flag) {
    if (threadIdx.x == 0) atomicExch(P.status, FF_ERR_TIMEOUT | 0x400);   // low byte: status, next byte: which kernel
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tm, 512);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 5-D map over a [slices][T][n][n][128] bf16 grid; box = 128/n whole lines along w (along_w) or one
// line along h.
bool encode_wh_map(CUtensorMap* map, const void* base, int n, int T, int slices, bool along_w) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", (void**)&enc, cudaEnableDefault, &qr) != cudaSuccess || !enc)
      return false;
  }
  cuuint64_t dims[5] = {(cuuint64_t)CH, (cuuint64_t)n, (cuuint64_t)n, (cuuint64_t)T, (cuuint64_t)slices};
  cuuint64_t strides[4] = {(cuuint64_t)CH * 2, (cuuint64_t)n * CH * 2, (cuuint64_t)n * n * CH * 2,
                           (cuuint64_t)T * n * n * CH * 2};
  cuuint32_t box[5] = {64, 1, 1, 1, 1};
  if (along_w) { box[1] = (cuuint32_t)n; box[2] = (cuuint32_t)(TILE_ROWS / n); } else { box[2] = (cuuint32_t)n; }
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Store map: the box of one epilogue warp, 32 channels of 32 consecutive positions along w
// (along_w) or along h, 64-byte swizzle.
bool encode_wh_store_map(CUtensorMap* map, const void* base, int n, int T, int slices, bool along_w) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", (void**)&enc, cudaEnableDefault, &qr) != cudaSuccess || !enc)
      return false;
  }
  cuuint64_t dims[5] = {(cuuint64_t)CH, (cuuint64_t)n, (cuuint64_t)n, (cuuint64_t)T, (cuuint64_t)slices};
  cuuint64_t strides[4] = {(cuuint64_t)CH * 2, (cuuint64_t)n * CH * 2, (cuuint64_t)n * n * CH * 2,
                           (cuuint64_t)T * n * n * CH * 2};
  cuuint32_t box[5] = {32, 1, 1, 1, 1};
  box[along_w ? 1 : 2] = 32;
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// bf16, head_dim 128, square h x w slabs whose side is a power of two in 32..128 (an epilogue
// warp's 32 rows must lie on one line).
bool ffk_dct_wh_supported(const FFDims& dm) {
  const int n = dm.W;
  return !dm.fp32 && dm.d == CH && dm.H == dm.W && (n == 32 || n == 64 || n == 128);
}

// Can a group of `g` tensor-heads run fused on a grid of `sm_count` CTAs?  The second pass must
// trail by the full lag, and no tile may wait for a counter whose release is deferred behind it.
bool ffk_dct_wh_usable(const FFDims& dm, int g, int sm_count) {
  if (!ffk_dct_wh_supported(dm)) return false;
  int ring, lag;
  ffk_dct_wh_shape(dm, &ring, &lag);
  const int tps = dm.W * dm.W / TILE_ROWS;
  return g * dm.T >= lag && (long long)lag * 2 * tps > sm_count + tps;
}

// Ring depth and lag: the second pass trails the first by about three rounds of the grid, and the
// ring is twice that deep, so neither dependency normally has to be waited for.
void ffk_dct_wh_shape(const FFDims& dm, int* ring, int* lag) {
  const int tps = dm.W * dm.W / TILE_ROWS;
  int D = (3 * 160 + 2 * tps - 1) / (2 * tps) + 1;
  *lag = D;
  *ring = 2 * D + 2;
}

size_t ffk_dct_wh_scratch_bytes(const FFDims& dm, int group) {
  int ring, lag;
  ffk_dct_wh_shape(dm, &ring, &lag);
  const size_t slab = (size_t)dm.H * dm.W * CH * 2;
  return 2 * ring * slab + (((size_t)2 * group * dm.T * sizeof(int)) + 255) / 256 * 256;
}

// One fused launch over `g` tensor-heads.  forward: src0..2 = Q, K, V (the caller's tensors), first
// tensor-head index g0 = tensor * BH + bh, result in out_hi/out_lo ([g][T][H][W][128]) and `side`.
// inverse: src0, src1 = hi/lo grids ([g][T][H][W][128]), g0 = first head, result in out_hi = the
// caller's out tensor.  `ring` holds 2 * ring * slab bytes followed by the counters.
cudaError_t ffk_dct_wh_launch(ff_plan* p, int forward, const void* src0, const void* src1, const void* src2, int g0, int g,
                              void* ring, void* out_hi, void* out_lo, float* side, cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int n = dm.W;
  WhParams P{};
  P.dm = dm; P.n = n; P.forward = forward; P.group = g; P.group_start = g0;
  ffk_dct_wh_shape(dm, &P.ring, &P.lag);
  const int S = g * dm.T;
  if (P.lag > S) P.lag = S;
  const size_t slab = (size_t)n * n * CH * 2;
  void* ring_hi = ring;                                  // [ring][H][W][128]
  void* ring_lo = (char*)ring + (size_t)P.ring * slab;
  P.cnt_a = (int*)((char*)ring + 2 * (size_t)P.ring * slab);
  P.cnt_b = P.cnt_a + S;
  P.side = side; P.status = p->buf.status;
  // one image serves both passes: I kron C (forward) or I kron C^T (inverse) of the w axis
  P.image = p->dct_images + (size_t)(2 * ((forward ? 0 : 3) + 2)) * TILE_BYTES;
  cudaError_t e = cudaMemsetAsync(P.cnt_a, 0, (size_t)2 * S * sizeof(int), st);
  if (e != cudaSuccess) return e;
  if (!ffk_dct_wh_usable(dm, g, p->sm_count)) return cudaErrorInvalidValue;
  CUtensorMap m0, m1, m2, m3, m4, s_rh, s_rl, s_oh, s_ol;
  bool ok;
  if (forward)
    ok = encode_wh_map(&m0, src0, n, dm.T, dm.BH, true) && encode_wh_map(&m1, src1, n, dm.T, dm.BH, true) &&
         encode_wh_map(&m2, src2, n, dm.T, dm.BH, true) && encode_wh_map(&m3, ring_hi, n, P.ring, 1, false) &&
         encode_wh_map(&m4, ring_lo, n, P.ring, 1, false) &&
         encode_wh_store_map(&s_rh, ring_hi, n, P.ring, 1, true) && encode_wh_store_map(&s_rl, ring_lo, n, P.ring, 1, true) &&
         encode_wh_store_map(&s_oh, out_hi, n, dm.T, g, false) && encode_wh_store_map(&s_ol, out_lo, n, dm.T, g, false);
  else
    ok = encode_wh_map(&m0, src0, n, dm.T, g, false) && encode_wh_map(&m1, src1, n, dm.T, g, false) &&
         encode_wh_map(&m2, src1, n, dm.T, g, false) && encode_wh_map(&m3, ring_hi, n, P.ring, 1, true) &&
         encode_wh_map(&m4, ring_lo, n, P.ring, 1, true) &&
         encode_wh_store_map(&s_rh, ring_hi, n, P.ring, 1, false) && encode_wh_store_map(&s_rl, ring_lo, n, P.ring, 1, false) &&
         encode_wh_store_map(&s_oh, out_hi, n, dm.T, dm.BH, true) && encode_wh_store_map(&s_ol, out_hi, n, dm.T, dm.BH, true);
  if (!ok) return cudaErrorInvalidValue;
  const size_t smem = NSTAGE * STAGE_BYTES + 2 * TILE_BYTES + sizeof(WhShared) + 1024;
  e = cudaFuncSetAttribute(dct_wh_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int total = 2 * S * (n * n / TILE_ROWS);
  const int grid = total < p->sm_count ? total : p->sm_count;
  dct_wh_kernel<<<grid, WH_THREADS, smem, st>>>(m0, m1, m2, m3, m4, s_rh, s_rl, s_oh, s_ol, P);
  p->launches += 1;
  return cudaGetLastError();
}
