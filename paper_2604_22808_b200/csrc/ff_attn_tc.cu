// Band attention on the 5th-generation tensor cores ("Hierarchical frequency-domain attention":
// strided block-sparse attention on the mid band, sliding-window attention on the high band, and
// dense attention on the pooled low band when that is at least a tile long), bf16 operands, fp32
// accumulation, head_dim 128 or 64 (template parameter HD).
//
// One persistent launch runs both branches from a worklist of (head, band, pair of query tiles)
// items that is rebuilt from the head-to-band allocation before every launch.  A CTA owns every
// gridDim-th item.  An item is two neighbouring 128-row query tiles ("streams" A and B) that walk
// one sequence of 128-key tiles together: both streams of a mid-band item see every key tile of
// their residue class; in the high band the union of the two windows is 2 + 2R/128 key tiles of
// which each stream takes part in 1 + 2R/128.  K and V tiles are therefore fetched once for two
// query tiles, and while the softmax warps of one stream work the tensor core runs the other's MMAs.
//   warp 0       TMA producer: the two Q tiles, K and V tiles (two stages each)
//   warp 1       tcgen05.mma issuer: S_x = Q_x K^T (operands from shared memory), O_x += P_x V
//                (A = P from tensor memory, B = V as an MN-major operand), issue order
//                PV_A[j], QK_A[j+1], PV_B[j], QK_B[j+1]; owns the tensor-memory allocation
//   warps 2..17  softmax: per stream two threads per query row (row = TMEM lane, 64 key columns
//                each); scores read with tcgen05.ld, key masks generated in registers from the row's
//                band rank, P written back to tensor memory as bf16 over the thread's own scores; O
//                accumulates in tensor memory and is rescaled only when a row maximum grows by > 2^8
// Tensor memory (512 columns): S/P of stream A, S/P of stream B, O of stream A, O of stream B.
// Every wait is bounded; when one runs out the CTA raises FF_ERR_TIMEOUT in the plan's status
// word, stops taking work, lets its copies drain, frees its tensor memory and returns.
#include <cuda.h>

#include "ff_internal.h"
#include "ff_sm100.cuh"

using namespace sm100;

namespace {

constexpr int TILE = 128;            // query rows per stream = key rows per tile
constexpr int HD_MAX = 128;          // largest head_dim; the shared-memory slots are sized for it
constexpr int TILE_BYTES = TILE * HD_MAX * 2;
constexpr int HALF_BYTES = TILE_BYTES / 2;
constexpr int MAX_UNITS = 1024;
constexpr int NSPLIT = 2;                // softmax threads per query row
constexpr int SCOLS = TILE / NSPLIT;     // key columns per softmax thread
constexpr int TC_THREADS = 64 + 2 * 128 * NSPLIT;   // TMA warp, MMA warp, 2 streams x 4 NSPLIT softmax warps
constexpr float LAZY_LOG2 = 8.0f;    // rescale O only when the running max grows by more than this (log2 units)

struct TcParams {
  FFDims dm;
  const uint8_t* alloc;
  int* work;          // [0] = number of units, [1] = total items, then offsets[MAX_UNITS+1], desc[MAX_UNITS], tiles[MAX_UNITS]
  __nv_bfloat16* y_mid;
  __nv_bfloat16* y_high;
  float* y_low;       // [BH][Nbar][d] fp32, written when low_on
  int low_on;         // heads whose mask has the low band run it here (band code 0: dense over Nbar pooled tokens)
  int* status;
  int rb_mid;         // rows per TMA box of the mid map = min(b, 128)
};

// The residue classes of the mid band come in two sizes: the first `rem` = nb mod s classes hold
// one block more than the others.  Items of a (head, mid band) unit are numbered class by class.
struct MidShape {
  int rem;              // classes with the larger block count
  int nclass;           // residue classes that exist: min(nb, s)
  int nt_big, nt_small; // query (= key) tiles of a class of either size
  int pairs_big, pairs_small;
  int items;            // items of one head's mid band
};

__host__ __device__ __forceinline__ MidShape mid_shape(const FFDims& dm) {
  MidShape m;
  const long long q = dm.s > 0 ? dm.nb / dm.s : 0;
  m.rem = dm.s > 0 ? (int)(dm.nb % dm.s) : 0;
  m.nclass = (int)(dm.nb < dm.s ? dm.nb : dm.s);
  m.nt_big = (int)(((q + 1) * dm.b + TILE - 1) / TILE);
  m.nt_small = (int)((q * dm.b + TILE - 1) / TILE);
  m.pairs_big = (m.nt_big + 1) / 2;
  m.pairs_small = (m.nt_small + 1) / 2;
  m.items = m.rem * m.pairs_big + (m.nclass - m.rem) * m.pairs_small;
  return m;
}

// Worklist: one unit per (head, mid band) and per (head, high band) that the allocation executes;
// mid units first (their items are the long ones).  An item is a pair of query tiles.
__global__ void build_worklist_kernel(TcParams P) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  const FFDims& dm = P.dm;
  int* offsets = P.work + 2;
  int* desc = offsets + MAX_UNITS + 1;
  int* tiles = desc + MAX_UNITS;
  int nu = 0, total = 0;
  const MidShape ms = mid_shape(dm);
  if (P.low_on) {
    const int nt = (int)((dm.Nbar + TILE - 1) / TILE);
    for (int bh = 0; bh < dm.BH && nu < MAX_UNITS; ++bh) {
      if (!(P.alloc[bh] & FF_BAND_LOW)) continue;
      offsets[nu] = total; desc[nu] = (bh << 12); tiles[nu] = nt;
      total += (nt + 1) / 2; ++nu;
    }
  }
  // (the anchor pattern of the mid band is not a union of dense classes: those heads run on the generic kernel)
  for (int bh = 0; bh < dm.BH && nu < MAX_UNITS && dm.pattern == FF_MID_STRIDED; ++bh) {
    if (!(P.alloc[bh] & FF_BAND_MID)) continue;
    offsets[nu] = total; desc[nu] = (bh << 12) | (1 << 10); tiles[nu] = 0;
    total += ms.items; ++nu;
  }
  for (int bh = 0; bh < dm.BH && nu < MAX_UNITS; ++bh) {
    if (!(P.alloc[bh] & FF_BAND_HIGH)) continue;
    const int nt = (int)((dm.Nhigh + TILE - 1) / TILE);
    offsets[nu] = total; desc[nu] = (bh << 12) | (2 << 10); tiles[nu] = nt;
    total += (nt + 1) / 2; ++nu;
  }
  offsets[nu] = total;
  P.work[0] = nu;
  P.work[1] = total;
}

struct Item {
  int band, bh, c;
  int tile_a;         // query tile of stream A; stream B takes tile_a + 1
  int has_b;          // stream B exists
  int nk;             // key tiles of the item
  long long n;        // band length
  long long ks;       // high: first key rank of key tile 0
};

struct Shared {
  uint64_t q_full, q_empty, k_full[2], k_empty[2], v_full[2], v_empty[2];
  uint64_t s_full[2], p_full[2], o_full[2], o_empty[2];      // per stream
  uint32_t tmem_base;
  int abort_flag;
  int n_units, total;
  MidShape ms;        // kept here rather than in every thread's registers
  int offsets[MAX_UNITS + 1];
  int desc[MAX_UNITS];
  int ntile[MAX_UNITS];
  // hand-shake slots of the threads of a row: (sequence number << 32) | float bits
  unsigned long long xmax[2][2][NSPLIT][128];     // [parity][stream][part][row]
  unsigned long long xsum[2][2][NSPLIT][128];
};

template <bool HAS_LOW>
__device__ __forceinline__ Item decode_item(const Shared& sh, const FFDims& dm, int it) {
  const MidShape& ms = sh.ms;
  int lo = 0, hi = sh.n_units - 1;
  while (lo < hi) {                       // last unit whose offset <= it
    const int mid = (lo + hi + 1) >> 1;
    if (sh.offsets[mid] <= it) lo = mid; else hi = mid - 1;
  }
  Item x;
  const int dsc = sh.desc[lo];
  x.bh = dsc >> 12; x.band = (dsc >> 10) & 3; x.c = 0;
  const int local = it - sh.offsets[lo];
  if (x.band == 1) {
    int pr, nt;
    if (local < ms.rem * ms.pairs_big) { x.c = local / ms.pairs_big; pr = local % ms.pairs_big; nt = ms.nt_big; }
    else {
      const int l2 = local - ms.rem * ms.pairs_big;
      x.c = ms.rem + l2 / ms.pairs_small; pr = l2 % ms.pairs_small; nt = ms.nt_small;
    }
    x.tile_a = 2 * pr;
    x.has_b = x.tile_a + 1 < nt;
    x.n = dm.Nmid;
    x.nk = nt;                            // every query tile of a class sees all its key tiles
    x.ks = 0;
  } else if (HAS_LOW && x.band == 0) {
    x.tile_a = 2 * local;
    x.has_b = x.tile_a + 1 < sh.ntile[lo];
    x.n = dm.Nbar;
    x.nk = sh.ntile[lo];                  // dense: every query tile sees every key tile
    x.ks = 0;
  } else {
    x.tile_a = 2 * local;
    x.has_b = x.tile_a + 1 < sh.ntile[lo];
    x.n = dm.Nhigh;
    const long long q0 = (long long)x.tile_a * TILE;
    x.ks = q0 - dm.R > 0 ? q0 - dm.R : 0;
    long long ke = q0 + (x.has_b ? 2 : 1) * TILE + dm.R;
    if (ke > x.n) ke = x.n;
    x.nk = (int)((ke - x.ks + TILE - 1) / TILE);
  }
  return x;
}

// Does stream `sx` (0 = A, 1 = B) take part in key tile j of the item?  Mid band: always.  High
// band: when the tile meets the window of the stream's 128 query rows.
__device__ __forceinline__ bool stream_active(const Item& x, const FFDims& dm, int sx, int j) {
  if (sx == 1 && !x.has_b) return false;
  if (x.band != 2) return true;
  const long long t0 = x.ks + (long long)j * TILE;
  const long long q0 = (long long)(x.tile_a + sx) * TILE;
  return t0 <= q0 + TILE - 1 + dm.R && t0 + TILE - 1 >= q0 - dm.R && t0 < x.n;
}

// Band rank of class-local position u of residue class c (mid band).
// (32-bit arithmetic: positions and ranks stay below 2^32 for every supported size.)
__device__ __forceinline__ long long mid_rank(const FFDims& dm, int c, long long u) {
  const unsigned uu = (unsigned)u, b = (unsigned)dm.b;
  const unsigned blk = uu / b;
  return (long long)(((unsigned)c + blk * (unsigned)dm.s) * b + (uu - blk * b));
}

// Issues the TMA loads of one 128-row tile (two 64-column halves) into `dst`; the caller has
// already announced the bytes on `bar`.  `first` = class-local position (mid) or band rank (high).
// `halves` = head_dim / 64.
__device__ __forceinline__ void load_tile(uint8_t* dst, const CUtensorMap* map, uint64_t* bar, const FFDims& dm,
                                          const Item& x, int slice, long long first, int rb, int halves, int* status) {
  // (debug build) a tile starts inside its band (rows past the end are zero-filled by the copy); the bytes were
  // announced on `bar` already, so a refused copy ends in the bounded wait of its consumer, not in a fault
  if (!FF_DBG_OK(first >= 0 && first < x.n + TILE && slice >= 0, status, 1)) return;
  if (x.band != 1) {
    tma_load_3d(dst, map, bar, 0, (int)first, slice);
    if (halves > 1) tma_load_3d(dst + HALF_BYTES, map, bar, 64, (int)first, slice);
  } else {
    for (int i = 0; i < TILE / rb; ++i) {
      const long long row = mid_rank(dm, x.c, first + (long long)i * rb);
      // a block past the end of the band starts beyond the tensor: the copy fills zeros
      const int y = row < dm.Nmid ? (int)row : (int)dm.Nmid;
      tma_load_3d(dst + i * rb * 128, map, bar, 0, y, slice);
      if (halves > 1) tma_load_3d(dst + HALF_BYTES + i * rb * 128, map, bar, 64, y, slice);
    }
  }
}

// The NSPLIT softmax threads of a row share one float each: a thread publishes (seq, value) in its
// slot and reads the others' slots, waiting (bounded) until they carry the same sequence number.
// `slots` points at [NSPLIT][128] entries; MAX selects max, otherwise sum.
template <bool MAX>
__device__ __forceinline__ bool row_exchange(unsigned long long* slots, int part, int row, unsigned seq, float& v,
                                             volatile int* abort_flag) {
  *(volatile unsigned long long*)(slots + part * 128 + row) = ((unsigned long long)seq << 32) | __float_as_uint(v);
  float acc = v;
#pragma unroll
  for (int o = 1; o < NSPLIT; ++o) {
    const volatile unsigned long long* theirs = slots + ((part + o) % NSPLIT) * 128 + row;
    const long long t0 = clock64();
    while (true) {
      const unsigned long long w = *theirs;
      if ((unsigned)(w >> 32) == seq) {
        const float xv = __uint_as_float((unsigned)w);
        acc = MAX ? fmaxf(acc, xv) : acc + xv;
        break;
      }
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitLimitCycles) { *abort_flag = 1; return false; }
    }
  }
  v = acc;
  return true;
}

// max of three (one instruction on sm_100)
__device__ __forceinline__ float max3f(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// The kernel body.  QKV_MAPS = false: map_a / map_b cover the plan's mid / high coefficient buffers,
// which hold Q~, K~ and V~ of head bh in slices bh, BH + bh and 2 BH + bh.  QKV_MAPS = true (the entry
// point that allocates nothing): map_a, map_b, map_c are the caller's separate Q, K, V tensors of one
// band, head bh in slice bh.
// HAS_LOW: the worklist may hold low-band items (band code 0).
template <int HD, bool QKV_MAPS, bool HAS_LOW>
__device__ __forceinline__ void attention_tc_body(const CUtensorMap& map_a, const CUtensorMap& map_b,
                                                  const CUtensorMap& map_c, const TcParams& P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;                       // stream A, stream B: 2 x 32 KB
  uint8_t* sK = smem + 2 * TILE_BYTES;      // 2 stages x 32 KB
  uint8_t* sV = smem + 4 * TILE_BYTES;      // 2 stages x 32 KB
  Shared& sh = *(Shared*)(smem + 6 * TILE_BYTES);
  const FFDims& dm = P.dm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int HALVES = HD / 64;                  // 64-channel halves of a row
  constexpr int TB = TILE * HD * 2;                // bytes of one tile
  constexpr int OCOLS = HD / NSPLIT;               // output columns per softmax thread

  if (threadIdx.x == 0) {
    mbar_init(&sh.q_full, 1); mbar_init(&sh.q_empty, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sh.k_full[i], 1); mbar_init(&sh.k_empty[i], 1);
      mbar_init(&sh.v_full[i], 1); mbar_init(&sh.v_empty[i], 1);
      mbar_init(&sh.s_full[i], 1); mbar_init(&sh.p_full[i], 128 * NSPLIT);
      mbar_init(&sh.o_full[i], 1); mbar_init(&sh.o_empty[i], 128 * NSPLIT);
    }
    sh.abort_flag = 0;
    sh.n_units = P.work[0];
    sh.total = P.work[1];
    sh.ms = mid_shape(dm);
    fence_mbar_init();
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 2 * 2 * NSPLIT * 128; i += TC_THREADS) {
    (&sh.xmax[0][0][0][0])[i] = 0ull;
    (&sh.xsum[0][0][0][0])[i] = 0ull;
  }
  for (int i = threadIdx.x; i <= sh.n_units; i += TC_THREADS) {
    sh.offsets[i] = P.work[2 + i];
    if (i < sh.n_units) {
      sh.desc[i] = P.work[2 + MAX_UNITS + 1 + i];
      sh.ntile[i] = P.work[2 + MAX_UNITS + 1 + MAX_UNITS + i];
    }
  }
  if (warp == 1) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = sh.tmem_base;
  const int total = sh.total;
  volatile int* abort_flag = &sh.abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&map_a); tma_prefetch_desc(&map_b); tma_prefetch_desc(&map_c);
      int iter = 0; unsigned g = 0;
      bool ok = true;
      for (int it = blockIdx.x; it < total && ok; it += gridDim.x, ++iter) {
        const Item x = decode_item<HAS_LOW>(sh, dm, it);
        const CUtensorMap* map = x.band == 1 ? &map_a : (!HAS_LOW || x.band == 2 || QKV_MAPS ? &map_b : &map_c);
        const CUtensorMap* mapq = QKV_MAPS ? &map_a : map;
        const CUtensorMap* mapk = QKV_MAPS ? &map_b : map;
        const CUtensorMap* mapv = QKV_MAPS ? &map_c : map;
        const int slice_k = QKV_MAPS ? x.bh : dm.BH + x.bh, slice_v = QKV_MAPS ? x.bh : 2 * dm.BH + x.bh;
        const int rb = x.band == 1 ? P.rb_mid : TILE;
        if (iter >= 1) ok = mbar_wait(&sh.q_empty, (iter - 1) & 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(&sh.q_full, x.has_b ? 2 * TB : TB);
        load_tile(sQ, mapq, &sh.q_full, dm, x, x.bh, (long long)x.tile_a * TILE, rb, HALVES, P.status);
        if (x.has_b) load_tile(sQ + TILE_BYTES, mapq, &sh.q_full, dm, x, x.bh, (long long)(x.tile_a + 1) * TILE, rb, HALVES, P.status);
        for (int j = 0; j < x.nk && ok; ++j, ++g) {
          const int st = g & 1;
          const long long first = x.band == 2 ? x.ks + (long long)j * TILE : (long long)j * TILE;
          if (g >= 2) ok = mbar_wait(&sh.k_empty[st], ((g >> 1) - 1) & 1, abort_flag);
          if (!ok) break;
          mbar_arrive_expect_tx(&sh.k_full[st], TB);
          load_tile(sK + st * TILE_BYTES, mapk, &sh.k_full[st], dm, x, slice_k, first, rb, HALVES, P.status);
          if (g >= 2) ok = mbar_wait(&sh.v_empty[st], ((g >> 1) - 1) & 1, abort_flag);
          if (!ok) break;
          mbar_arrive_expect_tx(&sh.v_full[st], TB);
          load_tile(sV + st * TILE_BYTES, mapv, &sh.v_full[st], dm, x, slice_v, first, rb, HALVES, P.status);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_qk = idesc_bf16_f32(TILE, TILE, false, false);
      const uint32_t idesc_pv = idesc_bf16_f32(TILE, HD, false, true);
      int iter = 0; unsigned g = 0;
      unsigned cp[2] = {0, 0};          // P phases consumed per stream
      unsigned ce[2] = {0, 0};          // items seen per stream (for the O buffer hand-back)
      bool ok = true;
      // S_x = Q_x K[tile]^T; `last` = no further QK uses this K stage
      auto issue_qk = [&](int sx, unsigned gt, bool last, bool release_q) {
        const int st = gt & 1;
        const uint32_t qbase = smem_u32(sQ + sx * TILE_BYTES), kbase = smem_u32(sK + st * TILE_BYTES);
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) {
          const uint32_t off = (k >> 2) * HALF_BYTES + (k & 3) * 32;
          umma_ss(tm + sx * 128, smem_desc_sw128(qbase + off, 16, 1024), smem_desc_sw128(kbase + off, 16, 1024),
                  idesc_qk, k > 0 ? 1u : 0u);
        }
        umma_commit(&sh.s_full[sx]);
        if (last) umma_commit(&sh.k_empty[st]);
        if (release_q) umma_commit(&sh.q_empty);
      };
      // O_x (+)= P_x V[tile]
      auto issue_pv = [&](int sx, unsigned gt, bool first_of_item, bool last) -> bool {
        const int st = gt & 1;
        if (!mbar_wait(&sh.p_full[sx], cp[sx] & 1, abort_flag)) return false;
        ++cp[sx];
        if (first_of_item && ce[sx] >= 1 && !mbar_wait(&sh.o_empty[sx], (ce[sx] - 1) & 1, abort_flag)) return false;
        tc_fence_after();
        const uint32_t vbase = smem_u32(sV + st * TILE_BYTES);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          // P of keys 16k..16k+15 sits at the start of the score columns of the thread that owns them
          const uint32_t pcol = ((16 * k) / SCOLS) * SCOLS + ((16 * k) % SCOLS) / 2;
          umma_ts(tm + 256 + sx * 128, tm + sx * 128 + pcol, smem_desc_sw128(vbase + k * 2048, HALF_BYTES, 1024),
                  idesc_pv, (first_of_item && k == 0) ? 0u : 1u);
        }
        umma_commit(&sh.o_full[sx]);
        if (last) umma_commit(&sh.v_empty[st]);
        return true;
      };
      for (int it = blockIdx.x; it < total && ok; it += gridDim.x, ++iter) {
        const Item x = decode_item<HAS_LOW>(sh, dm, it);
        ok = mbar_wait(&sh.q_full, iter & 1, abort_flag);
        if (!ok) break;
        const unsigned g0 = g;
        bool started[2] = {false, false};
        // key tile 0: QK of both streams
        ok = mbar_wait(&sh.k_full[g0 & 1], (g0 >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        {
          const bool a0 = stream_active(x, dm, 0, 0), b0 = stream_active(x, dm, 1, 0);
          if (a0) issue_qk(0, g0, !b0, x.nk == 1 && !b0);
          if (b0) issue_qk(1, g0, true, x.nk == 1);
        }
        for (int j = 0; j < x.nk && ok; ++j) {
          const unsigned gt = g0 + j;
          const bool aj = stream_active(x, dm, 0, j), bj = stream_active(x, dm, 1, j);
          const bool more = j + 1 < x.nk;
          const bool an = more && stream_active(x, dm, 0, j + 1), bn = more && stream_active(x, dm, 1, j + 1);
          bool v_ready = false, k_ready = false;
          for (int sx = 0; sx < 2 && ok; ++sx) {
            const bool act = sx ? bj : aj, nxt = sx ? bn : an;
            if (act) {
              if (!v_ready) { ok = mbar_wait(&sh.v_full[gt & 1], (gt >> 1) & 1, abort_flag); v_ready = true; if (!ok) break; }
              const bool last_pv = sx == 1 || !bj;
              ok = issue_pv(sx, gt, !started[sx], last_pv);
              started[sx] = true;
              if (!ok) break;
            }
            if (nxt) {
              if (!k_ready) { ok = mbar_wait(&sh.k_full[(gt + 1) & 1], ((gt + 1) >> 1) & 1, abort_flag); k_ready = true; if (!ok) break; tc_fence_after(); }
              const bool last_qk = sx == 1 || !bn;
              issue_qk(sx, gt + 1, last_qk, last_qk && j + 2 == x.nk);
            }
          }
        }
        g = g0 + x.nk;
        ce[0] += 1;
        if (x.has_b) ce[1] += 1;
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax
    // Warps 2..9 serve stream A, 10..17 stream B.  Inside a stream the first four warps take key
    // columns 0..63 of their 32 rows, the next four columns 64..127 (a warp reaches the TMEM lanes
    // 32*(warp%4)..+31).  The threads of a row agree on the row maximum through a bounded
    // hand-shake in shared memory; each keeps the partial row sum of its own columns.
    const int quarter = warp & 3;
    const int sx = (warp - 2) / (4 * NSPLIT);
    const int part = ((warp - 2) >> 2) % NSPLIT;
    const int row = quarter * 32 + lane;
    const int col0 = part * SCOLS;                      // first key column of this thread
    const int ocol0 = part * OCOLS;                     // first output column of this thread
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t s_addr = tm + lane_addr + sx * 128;
    const uint32_t o_addr = tm + lane_addr + 256 + sx * 128 + ocol0;     // this thread's output columns
    const float sl2 = rsqrtf((float)HD) * 1.4426950408889634f;
    unsigned cs = 0;                  // key tiles this stream has processed (phases of s_full / p_full)
    unsigned co = 0;                  // phases of o_full consumed
    unsigned ci = 0;                  // items this stream has processed
    bool ok = true;
    for (int it = blockIdx.x; it < total && ok; it += gridDim.x) {
      const Item x = decode_item<HAS_LOW>(sh, dm, it);
      if (sx == 1 && !x.has_b) continue;
      const int tile = x.tile_a + sx;
      // band rank of this thread's query row
      const long long u_q = (long long)tile * TILE + row;
      const long long p = x.band == 1 ? mid_rank(dm, x.c, u_q) : u_q;
      float m_ref = -1e30f, l = 0.f;
      bool first = true;
      for (int j = 0; j < x.nk && ok; ++j) {
        if (!stream_active(x, dm, sx, j)) continue;
        // valid key columns [clo, chi] of this row in this tile
        int clo = 0, chi = TILE - 1;
        bool full;
        if (x.band == 1) {
          const long long u0 = (long long)j * TILE;
          // ranks grow with the class-local position, so the valid keys are a prefix; a class is a whole number
          // of blocks and blocks tile the 128 rows, so only its last tile can hold keys past the band end
          full = j + 1 < x.nk || mid_rank(dm, x.c, u0 + TILE - 1) < dm.Nmid;
          if (!full) {
            chi = -1;
            for (int cc = TILE - 1; cc >= 0; --cc)
              if (mid_rank(dm, x.c, u0 + cc) < dm.Nmid) { chi = cc; break; }
          }
        } else if (HAS_LOW && x.band == 0) {
          const long long left = x.n - (long long)j * TILE;     // pooled tokens from this tile on
          full = left >= TILE;
          if (!full) chi = (int)left - 1;
        } else {
          const long long t0 = x.ks + (long long)j * TILE;
          const long long q0 = (long long)tile * TILE;
          full = (t0 >= q0 + TILE - 1 - dm.R) && (t0 + TILE - 1 <= q0 + dm.R) && (t0 + TILE <= x.n);
          if (!full) {
            const long long lo = p - dm.R - t0, hi = (p + dm.R < x.n - 1 ? p + dm.R : x.n - 1) - t0;
            clo = lo > 0 ? (int)(lo < TILE ? lo : TILE) : 0;
            chi = hi < TILE - 1 ? (int)(hi < -1 ? -1 : hi) : TILE - 1;
          }
        }
        // (edge tiles) the valid columns of this thread's 32-column chunks as bit masks
        uint32_t vmask[SCOLS / 32];
#pragma unroll
        for (int c = 0; c < SCOLS / 32; ++c) {
          const int a = clo - (col0 + c * 32), b = chi - (col0 + c * 32);      // valid bits [a, b] of the chunk
          const uint32_t lo_m = a <= 0 ? 0xffffffffu : (a >= 32 ? 0u : 0xffffffffu << a);
          const uint32_t hi_m = b >= 31 ? 0xffffffffu : (b < 0 ? 0u : 0xffffffffu >> (31 - b));
          vmask[c] = lo_m & hi_m;
        }
        ok = __all_sync(0xffffffffu, mbar_wait(&sh.s_full[sx], cs & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        // first sweep over this thread's raw scores: the row maximum of its columns
        float tmax = -INFINITY;
        {
          // (both 32-column chunks are requested before the first is used: one tensor-memory latency instead of two)
          static_assert(SCOLS == 64, "the first sweep reads two chunks");
          uint32_t r0[32], r1[32];
          tmem_ld32(s_addr + col0, r0);
          tmem_ld32(s_addr + col0 + 32, r1);
          tmem_wait_ld();
          if (full) {
            float t1 = -INFINITY;                          // two chains
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              tmax = max3f(tmax, __uint_as_float(r0[i]), __uint_as_float(r0[i + 1]));
              t1 = max3f(t1, __uint_as_float(r1[i]), __uint_as_float(r1[i + 1]));
            }
            tmax = fmaxf(tmax, t1);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              if (vmask[0] & (1u << i)) tmax = fmaxf(tmax, __uint_as_float(r0[i]));
              if (vmask[1] & (1u << i)) tmax = fmaxf(tmax, __uint_as_float(r1[i]));
            }
          }
        }
        // row maximum over the row's threads (slots alternate with the tile parity, so a partner's
        // read of this tile cannot meet this thread's write of the next)
        ok = __all_sync(0xffffffffu, row_exchange<true>(&sh.xmax[cs & 1][sx][0][0], part, row, cs + 1, tmax, abort_flag));
        if (!ok) break;
        const float m_new = fmaxf(m_ref, tmax);
        const bool need = (m_new - m_ref) * sl2 > LAZY_LOG2;
        const float alpha = need ? ex2((m_ref - m_new) * sl2) : 1.f;
        // The phase of the previous PV of this stream is normally consumed at the end of this tile,
        // just before P is published, when it has long completed; only a row maximum that grew past
        // the lazy threshold needs it now, because O is then rescaled in place.  Every phase of the
        // barrier is awaited exactly once, in order (parity waits must not skip phases), and before
        // the arrival that lets the next PV be issued.  All threads of a row see the same `need`.
        bool waited_prev = false;
        if (!first && __any_sync(0xffffffffu, need)) {
          ok = __all_sync(0xffffffffu, mbar_wait(&sh.o_full[sx], co & 1, abort_flag));
          ++co;
          waited_prev = true;
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int c = 0; c < OCOLS / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(o_addr + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            tmem_st32(o_addr + c * 32, r);
          }
          tmem_wait_st();
        }
        if (need) { l *= alpha; m_ref = m_new; }
        // P = 2^(s*scale*log2e - m) as bf16 over the scores, partial row sum
        const float mb = m_ref * sl2;
        float2 sum2 = make_float2(0.f, 0.f);              // (two scores per FMA / add: packed fp32 instructions)
        const float2 sl22 = make_float2(sl2, sl2), nmb2 = make_float2(-mb, -mb);
#pragma unroll
        for (int c = 0; c < SCOLS / 32; ++c) {
          // second sweep: the scores again (tensor-memory reads are cheap; keeping them in registers
          // is not, with 576 threads per CTA), P written over them
          uint32_t r[32];
          tmem_ld32(s_addr + col0 + c * 32, r);
          tmem_wait_ld();
          uint32_t pk[16];
          if (full) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float2 arg = __ffma2_rn(make_float2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1])), sl22, nmb2);
              const float2 pp = make_float2(ex2(arg.x), ex2(arg.y));
              sum2 = __fadd2_rn(sum2, pp);
              const __nv_bfloat162 v = __floats2bfloat162_rn(pp.x, pp.y);
              pk[i] = *(const uint32_t*)&v;
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float2 arg = __ffma2_rn(make_float2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1])), sl22, nmb2);
              float p0 = ex2(arg.x);
              float p1 = ex2(arg.y);
              if (!(vmask[c] & (1u << (2 * i)))) p0 = 0.f;
              if (!(vmask[c] & (2u << (2 * i)))) p1 = 0.f;
              sum2 = __fadd2_rn(sum2, make_float2(p0, p1));
              const __nv_bfloat162 v = __floats2bfloat162_rn(p0, p1);
              pk[i] = *(const uint32_t*)&v;
            }
          }
          tmem_st16(s_addr + col0 + c * 16, pk);      // inside this thread's own score columns
        }
        l += sum2.x + sum2.y;
        tmem_wait_st();
        if (!first && !waited_prev) {
          ok = __all_sync(0xffffffffu, mbar_wait(&sh.o_full[sx], co & 1, abort_flag));
          ++co;
          if (!ok) break;
        }
        tc_fence_before();
        mbar_arrive(&sh.p_full[sx]);
        first = false;
        ++cs;
      }
      if (!ok) break;
      // epilogue: O / l -> Y, once the item's last PV has landed; l = the partial row sums together
      ok = __all_sync(0xffffffffu, row_exchange<false>(&sh.xsum[ci & 1][sx][0][0], part, row, ci + 1, l, abort_flag));
      if (!ok) break;
      ok = __all_sync(0xffffffffu, mbar_wait(&sh.o_full[sx], co & 1, abort_flag));
      ++co;
      if (!ok) break;
      tc_fence_after();
      const float inv = 1.f / l;
      const bool store = p < x.n && FF_DBG_OK(p >= 0 && x.bh >= 0 && x.bh < dm.BH, P.status, 1);
      __nv_bfloat16* y = (x.band == 1 ? P.y_mid : P.y_high) + ((size_t)x.bh * x.n + (store ? p : 0)) * HD + ocol0;
      float* yl = HAS_LOW && x.band == 0 ? P.y_low + ((size_t)x.bh * x.n + (store ? p : 0)) * HD + ocol0 : nullptr;   // low band: fp32
#pragma unroll
      for (int c = 0; c < OCOLS / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(o_addr + c * 32, r);
        tmem_wait_ld();
        if (store && yl) {
#pragma unroll
          for (int v4 = 0; v4 < 8; ++v4)
            *(float4*)(yl + c * 32 + v4 * 4) = make_float4(__uint_as_float(r[v4 * 4]) * inv, __uint_as_float(r[v4 * 4 + 1]) * inv,
                                                           __uint_as_float(r[v4 * 4 + 2]) * inv, __uint_as_float(r[v4 * 4 + 3]) * inv);
        } else if (store) {
#pragma unroll
          for (int v4 = 0; v4 < 4; ++v4) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(r[v4 * 8 + 2 * i]) * inv,
                                                             __uint_as_float(r[v4 * 8 + 2 * i + 1]) * inv);
              w[i] = *(const uint32_t*)&v;
            }
            *(uint4*)(y + c * 32 + v4 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(&sh.o_empty[sx]);
      ++ci;
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (sh.abort_flag) {
    if (threadIdx.x == 0) atomicExch(P.status, FF_ERR_TIMEOUT | 0x100);   // low byte: status, next byte: which kernel
    // let copies that were already issued land before the shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tm, 512);
  }
}

template <int HD, bool HAS_LOW>
__global__ void __launch_bounds__(TC_THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_mid, const __grid_constant__ CUtensorMap map_high,
                    const __grid_constant__ CUtensorMap map_low,
                    const TcParams P) {
  attention_tc_body<HD, false, HAS_LOW>(map_mid, map_high, map_low, P);
}

// Same kernel on the caller's separate Q, K, V tensors of one band (see ff_high_attention_noalloc).
__global__ void __launch_bounds__(TC_THREADS, 1)
attention_tc_qkv_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                        const __grid_constant__ CUtensorMap map_v, const TcParams P) {
  attention_tc_body<HD_MAX, true, false>(map_q, map_k, map_v, P);
}

// Scratch of ff_high_attention_noalloc: the worklist, one band mask per head and a status word.
// 13,824 bytes in every GPU context that loads this library, held until the process exits.
constexpr int NOALLOC_MAX_HEADS = MAX_UNITS;
constexpr size_t NOALLOC_WORK_BYTES = ((2 + 3 * MAX_UNITS + 1) * sizeof(int) + 255) / 256 * 256;
constexpr size_t NOALLOC_BYTES = NOALLOC_WORK_BYTES + NOALLOC_MAX_HEADS + 256;
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_BYTES];

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool encode_band_map(CUtensorMap* map, void* base, long long rows, int slices, int box_rows, int hd = HD_MAX) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", (void**)&enc, cudaEnableDefault, &qr) != cudaSuccess || !enc)
      return false;
  }
  cuuint64_t dims[3] = {(cuuint64_t)hd, (cuuint64_t)rows, (cuuint64_t)slices};
  cuuint64_t strides[2] = {(cuuint64_t)hd * 2, (cuuint64_t)rows * hd * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

size_t ffk_tc_work_bytes() { return (size_t)(2 + 3 * MAX_UNITS + 1) * sizeof(int); }

// The tensor-core kernel covers bf16, head_dim 128 or 64 and block sizes that tile 128 rows evenly.
bool ffk_tc_supported(const FFDims& dm) {
  if (dm.fp32 || (dm.d != 128 && dm.d != 64)) return false;
  const bool b_ok = (dm.b <= TILE) ? (dm.b >= 8 && TILE % dm.b == 0) : (dm.b % TILE == 0);
  if (!b_ok) return false;
  if ((long long)dm.BH * 2 > MAX_UNITS || dm.BH >= (1 << 19)) return false;
  if ((long long)dm.BH * (mid_shape(dm).items + (dm.Nhigh + 2 * TILE - 1) / (2 * TILE)) >= (1LL << 31)) return false;
  if (dm.Nmid >= (1LL << 31) - 256 || dm.Nhigh >= (1LL << 31) - 256) return false;
  return true;
}

bool ffk_tc_prepare(ff_plan* p) {
  static_assert(sizeof(CUtensorMap) <= sizeof(p->tmap_mid), "tensor map storage too small");
  const FFDims& dm = p->dm;
  const int rb = dm.b < TILE ? dm.b : TILE;
  // (an empty mid band has no items; its map is encoded over one row of the high band's buffer and never used)
  if (!encode_band_map((CUtensorMap*)p->tmap_mid, dm.Nmid > 0 ? p->buf.spec_mid : p->buf.spec_high, dm.Nmid > 0 ? dm.Nmid : 1,
                       3 * dm.BH, dm.Nmid > 0 ? rb : 1, dm.d) ||
      !encode_band_map((CUtensorMap*)p->tmap_high, p->buf.spec_high, dm.Nhigh, 3 * dm.BH, TILE, dm.d))
    return false;
  // The low branch joins this launch when the pooled band is at least one tile long (shorter ones
  // stay on the generic fp32 kernel, which is exact and costs microseconds there).
  p->low_tc_ok = p->buf.pooled_bf && dm.Nbar >= TILE && dm.Nbar < (1LL << 31) - 256 && (long long)dm.BH * 3 <= MAX_UNITS &&
                 encode_band_map((CUtensorMap*)p->tmap_low, p->buf.pooled_bf, dm.Nbar, 3 * dm.BH, TILE, dm.d);
  return true;
}

cudaError_t ffk_attention_tc(ff_plan* p, cudaStream_t st) {
  const FFDims& dm = p->dm;
  TcParams P;
  P.dm = dm; P.alloc = p->buf.alloc; P.work = p->buf.work;
  P.y_mid = (__nv_bfloat16*)p->buf.y_mid; P.y_high = (__nv_bfloat16*)p->buf.y_high;
  P.y_low = p->buf.y_low; P.low_on = p->low_tc_ok ? 1 : 0;
  P.status = p->buf.status; P.rb_mid = dm.b < TILE ? dm.b : TILE;
  build_worklist_kernel<<<1, 32, 0, st>>>(P);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const size_t smem = 6 * TILE_BYTES + sizeof(Shared) + 1024;
  const CUtensorMap& mm = *(const CUtensorMap*)p->tmap_mid;
  const CUtensorMap& mh = *(const CUtensorMap*)p->tmap_high;
  const CUtensorMap& ml = p->low_tc_ok ? *(const CUtensorMap*)p->tmap_low : mh;
#define FF_ATT(D, LOW)                                                                                             \
  do {                                                                                                             \
    e = cudaFuncSetAttribute(attention_tc_kernel<D, LOW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    if (e == cudaSuccess) attention_tc_kernel<D, LOW><<<p->sm_count, TC_THREADS, smem, st>>>(mm, mh, ml, P);       \
  } while (0)
  if (dm.d == 128) { if (p->low_tc_ok) FF_ATT(128, true); else FF_ATT(128, false); }
  else { if (p->low_tc_ok) FF_ATT(64, true); else FF_ATT(64, false); }
#undef FF_ATT
  if (e != cudaSuccess) return e;
  p->launches += 2;
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// ff_high_attention_noalloc: the high-band operator for callers that cannot allocate.
// ------------------------------------------------------------------------------------------------
#include <mutex>

extern "C" ff_status_t ff_high_attention_noalloc(const void* q, const void* k, const void* v, void* y, int32_t heads,
                                                 int64_t n, int32_t radius, int32_t sync, void* cuda_stream) {
  if (!q || !k || !v || !y) { ff_set_thread_error("ff_high_attention_noalloc: a tensor pointer is NULL"); return FF_ERR_INVALID_ARG; }
  if ((((uintptr_t)q) | ((uintptr_t)k) | ((uintptr_t)v) | ((uintptr_t)y)) & 15) {
    ff_set_thread_error("ff_high_attention_noalloc: tensors must be 16-byte aligned");
    return FF_ERR_INVALID_ARG;
  }
  if (heads < 1 || n < 1 || radius < 0) {
    ff_set_thread_error("ff_high_attention_noalloc: need heads >= 1, n >= 1, radius >= 0");
    return FF_ERR_INVALID_ARG;
  }
  if (heads > NOALLOC_MAX_HEADS || n >= (1LL << 31) - 256) {
    ff_set_thread_error("ff_high_attention_noalloc: the built-in scratch covers at most 1024 heads and 2^31-257 tokens per head");
    return FF_ERR_UNSUPPORTED;
  }
  // the worklist counts items (pairs of 128-row query tiles) of all heads in 32 bits
  if ((long long)heads * ((n + 2 * TILE - 1) / (2 * TILE)) >= (1LL << 31)) {
    ff_set_thread_error("ff_high_attention_noalloc: heads x ceil(n / 256) must stay below 2^31");
    return FF_ERR_UNSUPPORTED;
  }
  // Device address of the scratch array, looked up once per device with that device current: in host
  // code the array's name is only a handle, not an address a kernel could use.
  static std::mutex mu;
  static unsigned char* dev_scratch[64] = {};
  static int sm_counts[64] = {};
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= 64) { ff_set_thread_error("ff_high_attention_noalloc: no usable current device"); return FF_ERR_CUDA; }
  unsigned char* scratch = nullptr;
  int sms = 0;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!dev_scratch[dev]) {
      void* ptr = nullptr;
      e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
      if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sm_counts[dev], cudaDevAttrMultiProcessorCount, dev);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(attention_tc_qkv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(6 * TILE_BYTES + sizeof(Shared) + 1024));
      if (e != cudaSuccess || !ptr) { ff_set_thread_error(cudaGetErrorString(e)); return FF_ERR_CUDA; }
      dev_scratch[dev] = (unsigned char*)ptr;
    }
    scratch = dev_scratch[dev];
    sms = sm_counts[dev];
  }
  CUtensorMap mq, mk, mv;
  if (!encode_band_map(&mq, const_cast<void*>(q), n, heads, TILE) || !encode_band_map(&mk, const_cast<void*>(k), n, heads, TILE) ||
      !encode_band_map(&mv, const_cast<void*>(v), n, heads, TILE)) {
    ff_set_thread_error("ff_high_attention_noalloc: could not encode the tensor maps");
    return FF_ERR_CUDA;
  }
  cudaStream_t st = (cudaStream_t)cuda_stream;
  TcParams P{};
  P.dm.B = 1; P.dm.heads = heads; P.dm.BH = heads; P.dm.d = HD_MAX; P.dm.R = radius;
  P.dm.Nhigh = n; P.dm.Nmid = 0; P.dm.nb = 0; P.dm.s = 1; P.dm.b = TILE; P.dm.r = 1;
  P.work = (int*)scratch;
  uint8_t* masks = scratch + NOALLOC_WORK_BYTES;
  P.alloc = masks;
  P.status = (int*)(scratch + NOALLOC_WORK_BYTES + NOALLOC_MAX_HEADS);
  P.y_mid = nullptr; P.y_high = (__nv_bfloat16*)y; P.rb_mid = TILE;
  // The array keeps the previous call's contents: rewrite the masks and clear the status word; the
  // worklist is rebuilt by its kernel.
  e = cudaMemsetAsync(masks, FF_BAND_HIGH, (size_t)heads, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(P.status, 0, sizeof(int), st);
  if (e == cudaSuccess) { build_worklist_kernel<<<1, 32, 0, st>>>(P); e = cudaGetLastError(); }
  if (e == cudaSuccess) {
    attention_tc_qkv_kernel<<<sms, TC_THREADS, 6 * TILE_BYTES + sizeof(Shared) + 1024, st>>>(mq, mk, mv, P);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) { ff_set_thread_error(cudaGetErrorString(e)); return FF_ERR_CUDA; }
  if (sync) {
    int word = 0;
    e = cudaMemcpyAsync(&word, P.status, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) { ff_set_thread_error(cudaGetErrorString(e)); return FF_ERR_CUDA; }
    if (word != 0) { ff_set_thread_error("ff_high_attention_noalloc: a bounded device-side wait expired"); return FF_ERR_TIMEOUT; }
  }
  return FF_OK;
}
