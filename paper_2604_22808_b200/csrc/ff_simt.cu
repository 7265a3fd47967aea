// Generic FP32-arithmetic kernels of the FreqFormer forward.  They cover every configuration the
// ABI accepts (any storage type, head_dim, block/stride/radius) and are the path of the fp32
// workload; the bf16 workloads replace the attention step with the tensor-core kernel.
#include "ff_internal.h"

namespace {

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T* p, float v);
template <> __device__ __forceinline__ void stf<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ------------------------------------------------------------------------------------------------
// One axis of the separable transform ("Separable spectral decomposition"):
//   out[o][a][c] = sum_b Mat[a][b] * in[o][b][c],   a, b in [0,n), c in [0,inner), o in [0,outer)
// with the tensor-head as the slowest index.  Mat is C (forward) or C^T (inverse).
// MODE 0: `in` is the caller's Q/K/V (storage type), `out` an fp32 scratch grid.
// MODE 1: fp32 scratch -> fp32 scratch.
// MODE 2: fp32 scratch -> band-major coefficient buffers (forward, last axis = t): the rank of
//         every coefficient is evaluated in registers from the nested-box closed form.
// MODE 3: fp32 scratch -> the caller's `out` tensor (storage type).
// ------------------------------------------------------------------------------------------------
constexpr int DCT_IC = 64;       // columns per CTA tile
constexpr int DCT_THREADS = 256;

struct DctPassParams {
  const void* src[3];   // MODE 0: Q, K, V; otherwise src[0] = scratch
  void* dst;            // MODE 0/1: scratch; MODE 3: out tensor
  const float* mat;     // [n][n]
  int n, inner, outer;
  int group_start;      // first tensor-head index of this launch
  int BH;
  long long N_d;        // elements per tensor-head
  // MODE 2
  FFDims dm;
  float* spec_low; void* spec_mid; void* spec_high;
};

template <typename ST, int MODE>
__global__ void __launch_bounds__(DCT_THREADS) dct_pass_kernel(const DctPassParams P) {
  extern __shared__ float smem[];
  const int n = P.n;
  const int npad = (n + 7) & ~7;
  float* matT = smem;                       // [b][npad]: matT[b][a] = Mat[a][b]
  float* tile = smem + (size_t)n * npad;    // [b][DCT_IC]
  const int chunks = (P.inner + DCT_IC - 1) / DCT_IC;
  const int o = blockIdx.x / chunks;
  const int c0 = (blockIdx.x % chunks) * DCT_IC;
  const int gi = blockIdx.y;                // tensor-head inside the group
  const int th = P.group_start + gi;        // global tensor-head index: tensor * BH + bh
  const int tid = threadIdx.x;

  for (int idx = tid; idx < n * npad; idx += DCT_THREADS) {
    const int b = idx / npad, a = idx % npad;
    matT[idx] = (a < n) ? P.mat[(size_t)a * n + b] : 0.f;
  }
  const size_t line0 = ((size_t)o * n) * P.inner + c0;
  if (MODE == 0) {
    const ST* src = (const ST*)P.src[th / P.BH] + (size_t)(th % P.BH) * P.N_d + line0;
    for (int idx = tid; idx < n * DCT_IC; idx += DCT_THREADS) {
      const int b = idx / DCT_IC, c = idx % DCT_IC;
      tile[idx] = (c0 + c < P.inner) ? ldf<ST>(src + (size_t)b * P.inner + c) : 0.f;
    }
  } else {
    const float* src = (const float*)P.src[0] + (size_t)gi * P.N_d + line0;
    for (int idx = tid; idx < n * DCT_IC; idx += DCT_THREADS) {
      const int b = idx / DCT_IC, c = idx % DCT_IC;
      tile[idx] = (c0 + c < P.inner) ? src[(size_t)b * P.inner + c] : 0.f;
    }
  }
  __syncthreads();

  const int agroups = npad / 8;
  for (int w = tid; w < agroups * (DCT_IC / 4); w += DCT_THREADS) {
    const int ag = w / (DCT_IC / 4), cg = w % (DCT_IC / 4);
    float acc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int b = 0; b < n; ++b) {
      const float4 x = *(const float4*)(tile + b * DCT_IC + cg * 4);
      const float4 m0 = *(const float4*)(matT + b * npad + ag * 8);
      const float4 m1 = *(const float4*)(matT + b * npad + ag * 8 + 4);
      const float mm[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
      const float xx[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(mm[i], xx[j], acc[i][j]);
    }
    const int c = c0 + cg * 4;
    if (c >= P.inner) continue;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int a = ag * 8 + i;
      if (a >= n) break;
      if (MODE == 0 || MODE == 1) {
        float* dst = (float*)P.dst + (size_t)gi * P.N_d + ((size_t)o * n + a) * P.inner + c;
        *(float4*)dst = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
      } else if (MODE == 3) {
        ST* dst = (ST*)P.dst + (size_t)th * P.N_d + ((size_t)o * n + a) * P.inner + c;
#pragma unroll
        for (int j = 0; j < 4; ++j) stf<ST>(dst + j, acc[i][j]);
      } else {  // MODE 2: a = k_t, column = (k_h, k_w, channel)
        const int d = P.dm.d;
        const int ch = c % d;
        const int kw = (c / d) % P.dm.W;
        const int kh = c / (d * P.dm.W);
        long long rank;
        const int band = ff_band_rank_of(P.dm, a, kh, kw, &rank);
        const int tensor = th / P.BH, bh = th % P.BH;
        if (band == 0) {
          float* dst = P.spec_low + (((size_t)tensor * P.BH + bh) * P.dm.Nlow + rank) * d + ch;
          *(float4*)dst = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
        } else {
          const long long nl = (band == 1) ? P.dm.Nmid : P.dm.Nhigh;
          ST* dst = (ST*)(band == 1 ? P.spec_mid : P.spec_high) + (((size_t)tensor * P.BH + bh) * nl + rank) * d + ch;
#pragma unroll
          for (int j = 0; j < 4; ++j) stf<ST>(dst + j, acc[i][j]);
        }
      }
    }
  }
}

template <typename ST, int MODE>
cudaError_t launch_dct_pass(const DctPassParams& P, int group, cudaStream_t st) {
  const int npad = (P.n + 7) & ~7;
  const size_t smem = ((size_t)P.n * npad + (size_t)P.n * DCT_IC) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(dct_pass_kernel<ST, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int chunks = (P.inner + DCT_IC - 1) / DCT_IC;
  dim3 grid((unsigned)((size_t)P.outer * chunks), (unsigned)group);
  dct_pass_kernel<ST, MODE><<<grid, DCT_THREADS, smem, st>>>(P);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Router statistics ("Spectral routing network"): sums of squared coefficients per sample, band
// and channel, pooled over heads, band ranks and the three tensors.
// ------------------------------------------------------------------------------------------------
constexpr int ENERGY_ROWS = 256;

template <typename ST>
__global__ void band_energy_kernel(const float* spec_low, const ST* spec_mid, const ST* spec_high, double* energy,
                                   FFDims dm) {
  const int band = blockIdx.y;
  const int th = blockIdx.z;                 // tensor * BH + bh
  const long long nl = band == 0 ? dm.Nlow : (band == 1 ? dm.Nmid : dm.Nhigh);
  const long long r0 = (long long)blockIdx.x * ENERGY_ROWS;
  if (r0 >= nl) return;
  const long long r1 = (r0 + ENERGY_ROWS < nl) ? r0 + ENERGY_ROWS : nl;
  const int d = dm.d;
  const int c = threadIdx.x % d;
  const int lane_rows = blockDim.x / d;
  const int sub = threadIdx.x / d;
  float acc = 0.f;
  if (sub < lane_rows) {
    for (long long r = r0 + sub; r < r1; r += lane_rows) {
      float v;
      if (band == 0) v = spec_low[((size_t)th * dm.Nlow + r) * d + c];
      else if (band == 1) v = ldf<ST>(spec_mid + ((size_t)th * dm.Nmid + r) * d + c);
      else v = ldf<ST>(spec_high + ((size_t)th * dm.Nhigh + r) * d + c);
      acc = fmaf(v, v, acc);
    }
    const int bh = th % dm.BH;
    const int sample = bh / dm.heads;
    atomicAdd(energy + ((size_t)sample * 3 + band) * d + c, (double)acc);
  }
}

// z = W2 relu(W1 [g; e(t)] + b1) + b2, pi = softmax(z), largest-remainder quota, one-hot masks.
__global__ void router_kernel(const double* energy, const float* timestep, const float* W1, const float* b1,
                              const float* W2, const float* b2, uint8_t* alloc, float* pi_out, FFDims dm) {
  extern __shared__ float sm[];
  const int d = dm.d, nin = 3 * d + dm.dt, hid = dm.hid;
  float* x = sm;            // [nin]
  float* h = sm + nin;      // [hid]
  __shared__ float z[3];
  const int sample = blockIdx.x;
  const long long cnt[3] = {dm.Nlow, dm.Nmid, dm.Nhigh};
  for (int i = threadIdx.x; i < 3 * d; i += blockDim.x) {
    const double terms = 3.0 * dm.heads * (double)(cnt[i / d] > 0 ? cnt[i / d] : 1);   // an empty band (two-band layer) has g = 0
    x[i] = (float)log1p(energy[(size_t)sample * 3 * d + i] / terms);
  }
  const int half = dm.dt / 2;
  const double t = (double)timestep[sample];
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    const double om = exp2(-(double)i / (double)half * 13.287712379549449);     // 10000^(-i/half); log2(10000)
    double sn, cs;
    sincos(t * om, &sn, &cs);
    x[3 * d + i] = (float)sn;
    x[3 * d + half + i] = (float)cs;
  }
  __syncthreads();
  // hidden layer: one warp per unit, lanes stride over the inputs (coalesced rows of W1)
  for (int j = threadIdx.x >> 5; j < hid; j += blockDim.x >> 5) {
    float acc = 0.f;
    for (int i = threadIdx.x & 31; i < nin; i += 32) acc = fmaf(W1[(size_t)j * nin + i], x[i], acc);
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) h[j] = fmaxf(acc + b1[j], 0.f);
  }
  __syncthreads();
  if (threadIdx.x < 3) {
    float acc = b2[threadIdx.x];
    for (int j = 0; j < hid; ++j) acc = fmaf(W2[threadIdx.x * hid + j], h[j], acc);
    z[threadIdx.x] = acc;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const float mx = fmaxf(z[0], fmaxf(z[1], z[2]));
    float e[3], pi[3];
    float sum = 0.f;
    for (int l = 0; l < 3; ++l) { e[l] = expf(z[l] - mx); sum += e[l]; }
    int base[3], total = 0;
    float frac[3];
    for (int l = 0; l < 3; ++l) {
      pi[l] = e[l] / sum;
      pi_out[sample * 3 + l] = pi[l];
      const float q = pi[l] * (float)dm.heads;
      base[l] = (int)floorf(q);
      frac[l] = q - floorf(q);
      total += base[l];
    }
    for (int left = dm.heads - total; left > 0; --left) {   // leftover heads: largest fraction, ties to the lower band
      int best = 0;
      for (int l = 1; l < 3; ++l) if (frac[l] > frac[best]) best = l;
      base[best] += 1;
      frac[best] = -1.f;
    }
    int hix = 0;
    for (int l = 0; l < 3; ++l)
      for (int k = 0; k < base[l] && hix < dm.heads; ++k) alloc[sample * dm.heads + hix++] = (uint8_t)(1 << l);
    for (; hix < dm.heads; ++hix) alloc[sample * dm.heads + hix] = FF_BAND_HIGH;
  }
}

// Low-band compression: mean over groups of r consecutive low ranks, for Q~, K~ and V~.
__global__ void pool_low_kernel(const float* spec_low, float* pooled, __nv_bfloat16* pooled_bf, FFDims dm) {
  // block = (d channels) x (POOL_ROWS pooled tokens)
  const long long g = (long long)blockIdx.x * blockDim.y + threadIdx.y;
  const int th = blockIdx.y;
  const int c = threadIdx.x;
  if (c >= dm.d || g >= dm.Nbar) return;
  const long long p0 = g * dm.r;
  const long long p1 = (p0 + dm.r < dm.Nlow) ? p0 + dm.r : dm.Nlow;
  float acc = 0.f;
  for (long long p = p0; p < p1; ++p) acc += spec_low[((size_t)th * dm.Nlow + p) * dm.d + c];
  const float v = acc / (float)(p1 - p0);
  pooled[((size_t)th * dm.Nbar + g) * dm.d + c] = v;
  if (pooled_bf) pooled_bf[((size_t)th * dm.Nbar + g) * dm.d + c] = __float2bfloat16_rn(v);
}

// ------------------------------------------------------------------------------------------------
// Band operators ("Hierarchical frequency-domain attention"), one warp per query row, online
// softmax with the score reduced by warp shuffles.  The key set of a row is generated from its
// rank: all pooled tokens (low), the blocks at block distance 0 mod s (mid), the window
// |p - p'| <= R (high).
// ------------------------------------------------------------------------------------------------
constexpr int ATT_WARPS = 8;

template <typename KT, int DPL>   // DPL = d / 32 channels per lane
__device__ __forceinline__ void attend_range(const KT* __restrict__ Kp, const KT* __restrict__ Vp, long long k0,
                                             long long k1, int d, const float (&q)[DPL], float scale, float& mx,
                                             float& den, float (&o)[DPL], int lane) {
  for (long long k = k0; k < k1; ++k) {
    const KT* kr = Kp + (size_t)k * d;
    float part = 0.f;
#pragma unroll
    for (int j = 0; j < DPL; ++j) part = fmaf(q[j], ldf<KT>(kr + lane + 32 * j), part);
    const float sc = warp_sum(part) * scale;
    const float nm = fmaxf(mx, sc);
    const float corr = expf(mx - nm);
    const float pr = expf(sc - nm);
    den = den * corr + pr;
    const KT* vr = Vp + (size_t)k * d;
#pragma unroll
    for (int j = 0; j < DPL; ++j) o[j] = fmaf(pr, ldf<KT>(vr + lane + 32 * j), o[j] * corr);
    mx = nm;
  }
}

template <typename ST, int DPL>
__global__ void __launch_bounds__(ATT_WARPS * 32) attention_simt_kernel(FFBuffers buf, FFDims dm, int band_bits) {
  const int band = blockIdx.z, bh = blockIdx.y;
  if (!(buf.alloc[bh] & band_bits & (1 << band))) return;
  const long long n = band == 0 ? dm.Nbar : (band == 1 ? dm.Nmid : dm.Nhigh);
  const long long p = (long long)blockIdx.x * ATT_WARPS + (threadIdx.x >> 5);
  if (p >= n) return;
  const int lane = threadIdx.x & 31;
  const int d = dm.d;
  const float scale = rsqrtf((float)d);
  float q[DPL], o[DPL];
  float mx = -INFINITY, den = 0.f;
#pragma unroll
  for (int j = 0; j < DPL; ++j) o[j] = 0.f;
  const size_t BHn = (size_t)dm.BH * n * d;   // one tensor's extent in this band's buffer
  if (band == 0) {
    const float* Qp = buf.pooled + (size_t)bh * n * d;
    const float* Kp = Qp + BHn;
    const float* Vp = Kp + BHn;
#pragma unroll
    for (int j = 0; j < DPL; ++j) q[j] = Qp[(size_t)p * d + lane + 32 * j];
    attend_range<float, DPL>(Kp, Vp, 0, n, d, q, scale, mx, den, o, lane);
    float* y = buf.y_low + ((size_t)bh * n + p) * d;
#pragma unroll
    for (int j = 0; j < DPL; ++j) y[lane + 32 * j] = o[j] / den;
  } else {
    const ST* Qp = (const ST*)(band == 1 ? buf.spec_mid : buf.spec_high) + (size_t)bh * n * d;
    const ST* Kp = Qp + BHn;
    const ST* Vp = Kp + BHn;
#pragma unroll
    for (int j = 0; j < DPL; ++j) q[j] = ldf<ST>(Qp + (size_t)p * d + lane + 32 * j);
    if (band == 1 && dm.pattern == FF_MID_ANCHOR) {
      // own block and every anchor block (block index = s-1 mod s)
      const long long J = p / dm.b;
      for (long long Jk = 0; Jk < dm.nb; ++Jk) {
        if (Jk != J && Jk % dm.s != dm.s - 1) continue;
        const long long k0 = Jk * dm.b;
        const long long k1 = (k0 + dm.b < n) ? k0 + dm.b : n;
        attend_range<ST, DPL>(Kp, Vp, k0, k1, d, q, scale, mx, den, o, lane);
      }
    } else if (band == 1) {
      const long long J = p / dm.b;
      for (long long Jk = J % dm.s; Jk < dm.nb; Jk += dm.s) {
        const long long k0 = Jk * dm.b;
        const long long k1 = (k0 + dm.b < n) ? k0 + dm.b : n;
        attend_range<ST, DPL>(Kp, Vp, k0, k1, d, q, scale, mx, den, o, lane);
      }
    } else {
      const long long k0 = (p - dm.R > 0) ? p - dm.R : 0;
      const long long k1 = (p + dm.R + 1 < n) ? p + dm.R + 1 : n;
      attend_range<ST, DPL>(Kp, Vp, k0, k1, d, q, scale, mx, den, o, lane);
    }
    ST* y = (ST*)(band == 1 ? buf.y_mid : buf.y_high) + ((size_t)bh * n + p) * d;
#pragma unroll
    for (int j = 0; j < DPL; ++j) stf<ST>(y + lane + 32 * j, o[j] / den);
  }
}

// ------------------------------------------------------------------------------------------------
// Working output of band `band` of head `bh` ("Cross-band residual exchange"): the operator's
// output where the head's mask has the band, the value coefficients V~ otherwise.
// ------------------------------------------------------------------------------------------------
template <typename ST>
struct BandView {
  const float* f32;   // low band rows (pooled output or V~ low)
  const ST* st;       // mid / high rows
  long long n;        // working length
  bool compressed;    // low band executed: row of rank p is p / r
};

template <typename ST>
__device__ __forceinline__ BandView<ST> band_view(const FFBuffers& buf, const FFDims& dm, int bh, int band) {
  BandView<ST> v;
  const bool exec = buf.alloc[bh] & (1 << band);
  const int d = dm.d;
  v.f32 = nullptr; v.st = nullptr; v.compressed = false;
  if (band == 0) {
    if (exec) { v.f32 = buf.y_low + (size_t)bh * dm.Nbar * d; v.n = dm.Nbar; v.compressed = true; }
    else { v.f32 = buf.spec_low + ((size_t)2 * dm.BH + bh) * dm.Nlow * d; v.n = dm.Nlow; }
  } else if (band == 1) {
    v.n = dm.Nmid;
    v.st = exec ? (const ST*)buf.y_mid + (size_t)bh * dm.Nmid * d
                : (const ST*)buf.spec_mid + ((size_t)2 * dm.BH + bh) * dm.Nmid * d;
  } else {
    v.n = dm.Nhigh;
    v.st = exec ? (const ST*)buf.y_high + (size_t)bh * dm.Nhigh * d
                : (const ST*)buf.spec_high + ((size_t)2 * dm.BH + bh) * dm.Nhigh * d;
  }
  return v;
}

// Summary tokens S = U_l Pool(Y^(l)): segment j covers [floor(j n/m), max(a+1, floor((j+1) n/m))).
// Two steps: segment sums (each segment split over several CTAs, 16-byte loads, partial sums
// added atomically into the summary buffer), then mean and projection in place.
constexpr int SUM_THREADS = 256;

template <typename ST>
__global__ void __launch_bounds__(SUM_THREADS) summary_partial_kernel(FFBuffers buf, FFDims dm, int split) {
  __shared__ float red[128];
  const int j = blockIdx.x / split, piece = blockIdx.x % split, band = blockIdx.y, bh = blockIdx.z;
  const int d = dm.d, vecs = d / 8;                // 8-channel vectors per row
  const BandView<ST> v = band_view<ST>(buf, dm, bh, band);
  if (v.n == 0) return;                            // empty band (two-band layer): no summary tokens
  const long long a = ((long long)j * v.n) / dm.m;
  long long e = ((long long)(j + 1) * v.n) / dm.m;
  if (e < a + 1) e = a + 1;
  const long long chunk = (e - a + split - 1) / split;
  const long long r0 = a + piece * chunk;
  const long long r1 = r0 + chunk < e ? r0 + chunk : e;
  const int vec = threadIdx.x % vecs, rsub = threadIdx.x / vecs, nrs = SUM_THREADS / vecs;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (rsub < nrs) {
    long long p = r0 + rsub;
    if (!v.f32 && sizeof(ST) == 2) {
      // bf16 rows, eight rows in flight per thread
      const __nv_bfloat16* base = (const __nv_bfloat16*)v.st + vec * 8;
      for (; p + 7 * nrs < r1; p += 8 * nrs) {
        uint4 x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = __ldcs((const uint4*)(base + (size_t)(p + u * nrs) * d));
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const uint32_t w[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            acc[2 * i] += __uint_as_float(w[i] << 16);
            acc[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
          }
        }
      }
    }
    for (; p < r1; p += nrs) {
      if (v.f32) {
        const float4 x0 = *(const float4*)(v.f32 + (size_t)p * d + vec * 8);
        const float4 x1 = *(const float4*)(v.f32 + (size_t)p * d + vec * 8 + 4);
        acc[0] += x0.x; acc[1] += x0.y; acc[2] += x0.z; acc[3] += x0.w;
        acc[4] += x1.x; acc[5] += x1.y; acc[6] += x1.z; acc[7] += x1.w;
      } else if (sizeof(ST) == 4) {
        const float4 x0 = *(const float4*)((const float*)v.st + (size_t)p * d + vec * 8);
        const float4 x1 = *(const float4*)((const float*)v.st + (size_t)p * d + vec * 8 + 4);
        acc[0] += x0.x; acc[1] += x0.y; acc[2] += x0.z; acc[3] += x0.w;
        acc[4] += x1.x; acc[5] += x1.y; acc[6] += x1.z; acc[7] += x1.w;
      } else {
        const uint4 x = *(const uint4*)((const __nv_bfloat16*)v.st + (size_t)p * d + vec * 8);
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          acc[2 * i] += __uint_as_float(w[i] << 16);
          acc[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
        }
      }
    }
  }
  // combine the row groups: channel sums through shared-memory atomics, then one global atomic per channel
  if (threadIdx.x < 128) red[threadIdx.x] = 0.f;
  __syncthreads();
  if (rsub < nrs) {
#pragma unroll
    for (int i = 0; i < 8; ++i) atomicAdd(&red[vec * 8 + i], acc[i]);
  }
  __syncthreads();
  if (threadIdx.x < d && r0 < r1)
    atomicAdd(buf.summary + (((size_t)bh * 3 + band) * dm.m + j) * d + threadIdx.x, red[threadIdx.x]);
}

template <typename ST>
__global__ void summary_finalize_kernel(FFBuffers buf, const float* U, FFDims dm, int identity_u) {
  __shared__ float pooled[128];
  const int j = blockIdx.x, band = blockIdx.y, bh = blockIdx.z;
  const int d = dm.d, c = threadIdx.x;
  const BandView<ST> v = band_view<ST>(buf, dm, bh, band);
  if (v.n == 0) return;                            // (its slots stay zero and are never attended)
  const long long a = ((long long)j * v.n) / dm.m;
  long long e = ((long long)(j + 1) * v.n) / dm.m;
  if (e < a + 1) e = a + 1;
  float* S = buf.summary + (((size_t)bh * 3 + band) * dm.m + j) * d;
  pooled[c] = S[c] / (float)(e - a);
  if (identity_u) { S[c] = pooled[c]; return; }
  __syncthreads();
  const float* Ul = U + ((size_t)band * d + c) * d;
  float s = 0.f;
  for (int i = 0; i < d; ++i) s = fmaf(Ul[i], pooled[i], s);
  S[c] = s;
}

// Exchange + recombination ("Cross-band residual exchange", "Reconstruction"): for every
// coefficient of the grid, fetch its band token, add softmax(y Z^T / sqrt(d)) Z over the 2m summary
// tokens of the other two bands, and write the row at its coefficient position (fp32 grid).
constexpr int EXC_WARPS = 8;

// Coefficients per warp: up to 8, fewer when the launch would otherwise have too few blocks.
static int exc_rounds(long long tokens, int g, int sm_count) {
  long long r = tokens * g / ((long long)EXC_WARPS * 8 * sm_count);
  return r < 1 ? 1 : (r > 8 ? 8 : (int)r);
}

template <typename ST, int DPL, typename OT>
__global__ void __launch_bounds__(EXC_WARPS * 32) exchange_recombine_kernel(FFBuffers buf, FFDims dm, int bh0,
                                                                             OT* grid_out, void* grid_lo, int low_only, int rounds) {
  extern __shared__ float S[];   // [3][m][d]
  const int gi = blockIdx.y, bh = bh0 + gi;
  const int d = dm.d, m = dm.m;
  for (int i = threadIdx.x; i < 3 * m * d; i += blockDim.x) S[i] = buf.summary[(size_t)bh * 3 * m * d + i];
  __syncthreads();
  // low_only: the launch covers the low band's coefficients only (the other bands are exchanged
  // by the tensor-core kernel); the index is then a low rank, unravelled inside the low box.
  const int lane = threadIdx.x & 31;
  // a block stages the summaries once and then works through rounds x EXC_WARPS coefficients
  for (int round = 0; round < rounds; ++round) {
  long long f = ((long long)blockIdx.x * rounds + round) * EXC_WARPS + (threadIdx.x >> 5);
  if (f >= (low_only ? dm.Nlow : dm.N)) return;
  int kw, kh, kt;
  if (low_only) {
    kw = (int)(f % dm.L[2]); kh = (int)((f / dm.L[2]) % dm.L[1]); kt = (int)(f / ((long long)dm.L[2] * dm.L[1]));
    f = ((long long)kt * dm.H + kh) * dm.W + kw;
  } else {
    kw = (int)(f % dm.W); kh = (int)((f / dm.W) % dm.H); kt = (int)(f / ((long long)dm.W * dm.H));
  }
  long long rank;
  const int band = ff_band_rank_of(dm, kt, kh, kw, &rank);
  const BandView<ST> v = band_view<ST>(buf, dm, bh, band);
  const long long row = v.compressed ? rank / dm.r : rank;
  float y[DPL], acc[DPL];
#pragma unroll
  for (int j = 0; j < DPL; ++j) {
    y[j] = v.f32 ? v.f32[(size_t)row * d + lane + 32 * j] : ldf<ST>(v.st + (size_t)row * d + lane + 32 * j);
    acc[j] = 0.f;
  }
  if (m > 0) {
    const float scale = rsqrtf((float)d);
    float mx = -INFINITY, den = 0.f;
    for (int ob = 0; ob < 3; ++ob) {
      if (ob == band || (ob == 1 && dm.Nmid == 0)) continue;     // own band; an empty mid band has no summaries
      for (int j2 = 0; j2 < m; ++j2) {
        const float* z = S + ((size_t)ob * m + j2) * d;
        float part = 0.f;
#pragma unroll
        for (int j = 0; j < DPL; ++j) part = fmaf(y[j], z[lane + 32 * j], part);
        const float sc = warp_sum(part) * scale;
        const float nm = fmaxf(mx, sc);
        const float corr = expf(mx - nm), pr = expf(sc - nm);
        den = den * corr + pr;
#pragma unroll
        for (int j = 0; j < DPL; ++j) acc[j] = fmaf(pr, z[lane + 32 * j], acc[j] * corr);
        mx = nm;
      }
    }
#pragma unroll
    for (int j = 0; j < DPL; ++j) acc[j] /= den;
  }
  // With a second grid (bf16 output) the value is stored in three bytes, rounded to 24 bits: its upper 16 bits
  // in grid_out, the next 8 bits in the byte grid.  A band's tokens share almost the same exchange offset, so a
  // single bf16 rounding would bias whole bands coherently and the inverse transform would focus that bias on a
  // few tokens.
  OT* dst = grid_out + ((size_t)gi * dm.N + f) * d;
#pragma unroll
  for (int j = 0; j < DPL; ++j) {
    const float v = y[j] + acc[j];
    if (grid_lo) {
      const uint32_t u = __float_as_uint(v) + 0x80u;
      ((uint16_t*)dst)[lane + 32 * j] = (uint16_t)(u >> 16);
      ((uint8_t*)grid_lo)[((size_t)gi * dm.N + f) * d + lane + 32 * j] = (uint8_t)(u >> 8);
    } else {
      stf<OT>(dst + lane + 32 * j, v);
    }
  }
  }
}

}  // namespace

// ================================================================================================
// Launchers
// ================================================================================================
template <typename ST>
static cudaError_t forward_transform_t(ff_plan* p, const void* Q, const void* K, const void* V, cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int total = 3 * dm.BH, G = p->lay.group;
  DctPassParams P{};
  P.BH = dm.BH; P.N_d = dm.N * dm.d; P.dm = dm;
  P.spec_low = p->buf.spec_low; P.spec_mid = p->buf.spec_mid; P.spec_high = p->buf.spec_high;
  for (int g0 = 0; g0 < total; g0 += G) {
    const int g = (total - g0 < G) ? total - g0 : G;
    P.group_start = g0;
    // w axis: lines of W elements with stride d
    P.src[0] = Q; P.src[1] = K; P.src[2] = V; P.dst = p->buf.scratchA; P.mat = p->basis[2];
    P.n = dm.W; P.inner = dm.d; P.outer = dm.T * dm.H;
    cudaError_t e = launch_dct_pass<ST, 0>(P, g, st);
    if (e != cudaSuccess) return e;
    // h axis
    P.src[0] = p->buf.scratchA; P.dst = p->buf.scratchB; P.mat = p->basis[1];
    P.n = dm.H; P.inner = dm.W * dm.d; P.outer = dm.T;
    e = launch_dct_pass<ST, 1>(P, g, st);
    if (e != cudaSuccess) return e;
    // t axis + band split
    P.src[0] = p->buf.scratchB; P.dst = nullptr; P.mat = p->basis[0];
    P.n = dm.T; P.inner = dm.H * dm.W * dm.d; P.outer = 1;
    e = launch_dct_pass<ST, 2>(P, g, st);
    if (e != cudaSuccess) return e;
    p->launches += 3;
  }
  return cudaSuccess;
}

cudaError_t ffk_forward_transform(ff_plan* p, const void* Q, const void* K, const void* V, cudaStream_t st) {
  return p->dm.fp32 ? forward_transform_t<float>(p, Q, K, V, st) : forward_transform_t<__nv_bfloat16>(p, Q, K, V, st);
}

cudaError_t ffk_band_energy(ff_plan* p, cudaStream_t st) {
  const FFDims& dm = p->dm;
  long long nmax = dm.Nhigh > dm.Nmid ? dm.Nhigh : dm.Nmid;
  if (dm.Nlow > nmax) nmax = dm.Nlow;
  dim3 grid((unsigned)((nmax + ENERGY_ROWS - 1) / ENERGY_ROWS), 3, (unsigned)(3 * dm.BH));
  const int threads = (256 / dm.d) * dm.d;
  if (dm.fp32)
    band_energy_kernel<float><<<grid, threads, 0, st>>>(p->buf.spec_low, (const float*)p->buf.spec_mid,
                                                        (const float*)p->buf.spec_high, p->buf.energy, dm);
  else
    band_energy_kernel<__nv_bfloat16><<<grid, threads, 0, st>>>(p->buf.spec_low, (const __nv_bfloat16*)p->buf.spec_mid,
                                                                (const __nv_bfloat16*)p->buf.spec_high, p->buf.energy, dm);
  p->launches += 1;
  return cudaGetLastError();
}

cudaError_t ffk_router(ff_plan* p, uint8_t* alloc_out, cudaStream_t st) {
  const FFDims& dm = p->dm;
  const size_t smem = (size_t)(3 * dm.d + dm.dt + dm.hid) * sizeof(float);
  router_kernel<<<dm.B, 256, smem, st>>>(p->buf.energy, p->buf.timestep, p->W1, p->b1, p->W2, p->b2, alloc_out,
                                         p->buf.pi, dm);
  p->launches += 1;
  return cudaGetLastError();
}

cudaError_t ffk_pool_low(ff_plan* p, cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int rows = dm.d <= 128 ? 512 / dm.d : 1;            // pooled tokens per CTA
  dim3 grid((unsigned)((dm.Nbar + rows - 1) / rows), (unsigned)(3 * dm.BH)), block((unsigned)dm.d, (unsigned)rows);
  pool_low_kernel<<<grid, block, 0, st>>>(p->buf.spec_low, p->buf.pooled, p->low_tc_ok ? p->buf.pooled_bf : nullptr, dm);
  p->launches += 1;
  return cudaGetLastError();
}

template <typename ST>
static cudaError_t attention_simt_t(ff_plan* p, int band_bits, cudaStream_t st) {
  const FFDims& dm = p->dm;
  long long nmax = 0;
  if ((band_bits & FF_BAND_LOW) && dm.Nbar > nmax) nmax = dm.Nbar;
  if ((band_bits & FF_BAND_MID) && dm.Nmid > nmax) nmax = dm.Nmid;
  if ((band_bits & FF_BAND_HIGH) && dm.Nhigh > nmax) nmax = dm.Nhigh;
  if (nmax == 0) return cudaSuccess;                 // (only an empty band was asked for)
  const int zdim = (band_bits & FF_BAND_HIGH) ? 3 : ((band_bits & FF_BAND_MID) ? 2 : 1);
  dim3 grid((unsigned)((nmax + ATT_WARPS - 1) / ATT_WARPS), (unsigned)dm.BH, zdim);
  switch (dm.d / 32) {
    case 1: attention_simt_kernel<ST, 1><<<grid, ATT_WARPS * 32, 0, st>>>(p->buf, dm, band_bits); break;
    case 2: attention_simt_kernel<ST, 2><<<grid, ATT_WARPS * 32, 0, st>>>(p->buf, dm, band_bits); break;
    case 3: attention_simt_kernel<ST, 3><<<grid, ATT_WARPS * 32, 0, st>>>(p->buf, dm, band_bits); break;
    default: attention_simt_kernel<ST, 4><<<grid, ATT_WARPS * 32, 0, st>>>(p->buf, dm, band_bits); break;
  }
  p->launches += 1;
  return cudaGetLastError();
}

cudaError_t ffk_attention_simt(ff_plan* p, int band_bits, cudaStream_t st) {
  return p->dm.fp32 ? attention_simt_t<float>(p, band_bits, st) : attention_simt_t<__nv_bfloat16>(p, band_bits, st);
}

cudaError_t ffk_summaries(ff_plan* p, cudaStream_t st) {
  const FFDims& dm = p->dm;
  cudaError_t e = cudaMemsetAsync(p->buf.summary, 0, (size_t)dm.BH * 3 * dm.m * dm.d * sizeof(float), st);
  if (e != cudaSuccess) return e;
  // split every segment so that each CTA reads about 1024 rows of the longest band
  long long longest = dm.Nhigh > dm.Nmid ? dm.Nhigh : dm.Nmid;
  int split = (int)((longest / dm.m + 1023) / 1024);
  if (split < 1) split = 1;
  if (split > 64) split = 64;
  dim3 pgrid((unsigned)(dm.m * split), 3, (unsigned)dm.BH), fgrid((unsigned)dm.m, 3, (unsigned)dm.BH);
  if (dm.fp32) {
    summary_partial_kernel<float><<<pgrid, SUM_THREADS, 0, st>>>(p->buf, dm, split);
    summary_finalize_kernel<float><<<fgrid, dm.d, 0, st>>>(p->buf, p->U, dm, p->identity_u);
  } else {
    summary_partial_kernel<__nv_bfloat16><<<pgrid, SUM_THREADS, 0, st>>>(p->buf, dm, split);
    summary_finalize_kernel<__nv_bfloat16><<<fgrid, dm.d, 0, st>>>(p->buf, p->U, dm, p->identity_u);
  }
  p->launches += 2;
  return cudaGetLastError();
}

__device__ __forceinline__ float exp2f_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Low band of the tensor-core inverse ("Cross-band residual exchange", "Reconstruction"): exchange + recombination
// of the low band's coefficients into the three-byte grids.  One warp per SOURCE row: a head that executes the
// low band has one pooled output row for every r consecutive coefficient ranks, so its update is computed once
// and written r times; other heads carry V~ low, one row per rank.  The scores of eight summaries at a time
// are reduced side by side (independent shuffle trees) and merged into the running softmax as a group
// (exponentials by ex2.approx on scores scaled to log2 units, like the tensor-core kernel's).  DPL = d / 32.
template <int DPL>
__global__ void __launch_bounds__(EXC_WARPS * 32) exchange_low_kernel(FFBuffers buf, FFDims dm, int bh0, __nv_bfloat16* grid_hi,
                                                                       uint8_t* grid_lo, int rounds) {
  extern __shared__ float S[];   // [3][m][d]
  const int gi = blockIdx.y, bh = bh0 + gi;
  const int d = dm.d, m = dm.m;
  for (int i = threadIdx.x; i < 3 * m * d; i += blockDim.x) S[i] = buf.summary[(size_t)bh * 3 * m * d + i];
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const bool exec = buf.alloc[bh] & FF_BAND_LOW;
  const float* src = exec ? buf.y_low + (size_t)bh * dm.Nbar * d : buf.spec_low + ((size_t)2 * dm.BH + bh) * dm.Nlow * d;
  const long long rows = exec ? dm.Nbar : dm.Nlow;
  const int rep = exec ? dm.r : 1;
  // the summaries of the other bands: the mid band's (none if it is empty), then the high band's
  const int k_first = dm.Nmid == 0 ? 2 * m : m, nkeys = 3 * m - k_first;
  const float scale = rsqrtf((float)d) * 1.4426950408889634f;      // scores in units of log2: exponentials by ex2
  for (int round = 0; round < rounds; ++round) {
    const long long row = ((long long)blockIdx.x * rounds + round) * EXC_WARPS + (threadIdx.x >> 5);
    if (row >= rows) return;
    float y[DPL], acc[DPL];
#pragma unroll
    for (int j = 0; j < DPL; ++j) { y[j] = src[(size_t)row * d + lane + 32 * j]; acc[j] = 0.f; }
    if (nkeys > 0) {
      float mx = -INFINITY, den = 0.f;
      for (int k0 = 0; k0 < nkeys; k0 += 8) {
        float sc[8];
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const float* z = S + (size_t)(k_first + (k0 + kk < nkeys ? k0 + kk : 0)) * d;
          float part = 0.f;
#pragma unroll
          for (int j = 0; j < DPL; ++j) part = fmaf(y[j], z[lane + 32 * j], part);
          sc[kk] = part;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) sc[kk] += __shfl_xor_sync(0xffffffffu, sc[kk], o);
        float nm = mx;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          sc[kk] = k0 + kk < nkeys ? sc[kk] * scale : -INFINITY;
          nm = fmaxf(nm, sc[kk]);
        }
        const float corr = exp2f_fast(mx - nm);
        den *= corr;
#pragma unroll
        for (int j = 0; j < DPL; ++j) acc[j] *= corr;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const float pr = exp2f_fast(sc[kk] - nm);         // (0 for the keys past the end)
          const float* z = S + (size_t)(k_first + (k0 + kk < nkeys ? k0 + kk : 0)) * d;
          den += pr;
#pragma unroll
          for (int j = 0; j < DPL; ++j) acc[j] = fmaf(pr, z[lane + 32 * j], acc[j]);
        }
        mx = nm;
      }
#pragma unroll
      for (int j = 0; j < DPL; ++j) acc[j] /= den;
    }
    // the value in three bytes (rounded to 24 bits: upper 16 bits and the next 8), at every rank the row stands for
    uint32_t u[DPL];
#pragma unroll
    for (int j = 0; j < DPL; ++j) u[j] = __float_as_uint(y[j] + acc[j]) + 0x80u;
    for (int i = 0; i < rep; ++i) {
      const long long p = row * rep + i;
      if (p >= dm.Nlow) break;
      const int kw = (int)(p % dm.L[2]), kh = (int)((p / dm.L[2]) % dm.L[1]), kt = (int)(p / ((long long)dm.L[2] * dm.L[1]));
      const size_t o = ((size_t)gi * dm.N + ((size_t)kt * dm.H + kh) * dm.W + kw) * d;
#pragma unroll
      for (int j = 0; j < DPL; ++j) {
        ((uint16_t*)grid_hi)[o + lane + 32 * j] = (uint16_t)(u[j] >> 16);
        grid_lo[o + lane + 32 * j] = (uint8_t)(u[j] >> 8);
      }
    }
  }
}

// Generic exchange + recombination into the hi/lo bf16 grids of the tensor-core inverse; DPL = d / 32.
template <int DPL>
static cudaError_t exchange_to_grids(ff_plan* p, long long tokens, int g, size_t smem, int h0, __nv_bfloat16* ghi,
                                     __nv_bfloat16* glo, int low_only, cudaStream_t st) {
  const int rounds = exc_rounds(tokens, g, p->sm_count);
  const long long per_block = (long long)EXC_WARPS * rounds;
  dim3 grid((unsigned)((tokens + per_block - 1) / per_block), (unsigned)g);
  cudaError_t e = cudaFuncSetAttribute(exchange_recombine_kernel<__nv_bfloat16, DPL, __nv_bfloat16>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  exchange_recombine_kernel<__nv_bfloat16, DPL, __nv_bfloat16><<<grid, EXC_WARPS * 32, smem, st>>>(p->buf, p->dm, h0, ghi, glo, low_only, rounds);
  return cudaGetLastError();
}

// Tensor-core inverse: exchange + recombination into a bf16 grid, then the three axis passes.
static cudaError_t exchange_inverse_tc(ff_plan* p, void* out, cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int G = p->dct_group;
  const size_t smem = (size_t)3 * dm.m * dm.d * sizeof(float);
  cudaError_t e = cudaSuccess;
  for (int h0 = 0; h0 < dm.BH; h0 += G) {
    const int g = (dm.BH - h0 < G) ? dm.BH - h0 : G;
    const size_t grid_bytes = ((size_t)G * dm.N * dm.d * 2 + 255) / 256 * 256;
    __nv_bfloat16* ghi = (__nv_bfloat16*)p->buf.scratchA;
    __nv_bfloat16* glo = (__nv_bfloat16*)((char*)p->buf.scratchA + grid_bytes);
    if (p->xtc_ok) {
      // mid and high bands on the tensor cores, the fp32 low band with its own kernel (one warp per source row)
      {
        const int rounds = exc_rounds(dm.Nlow, g, p->sm_count);
        const long long per_block = (long long)EXC_WARPS * rounds;
        dim3 grid((unsigned)((dm.Nlow + per_block - 1) / per_block), (unsigned)g);
        if (dm.d == 128) {
          e = cudaFuncSetAttribute(exchange_low_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
          if (e == cudaSuccess) exchange_low_kernel<4><<<grid, EXC_WARPS * 32, smem, st>>>(p->buf, dm, h0, ghi, (uint8_t*)glo, rounds);
        } else {
          e = cudaFuncSetAttribute(exchange_low_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
          if (e == cudaSuccess) exchange_low_kernel<2><<<grid, EXC_WARPS * 32, smem, st>>>(p->buf, dm, h0, ghi, (uint8_t*)glo, rounds);
        }
        if (e == cudaSuccess) e = cudaGetLastError();
      }
      if (e == cudaSuccess) e = ffk_exchange_tc(p, h0, g, ghi, glo, st);
    } else {
      e = dm.d == 128 ? exchange_to_grids<4>(p, dm.N, g, smem, h0, ghi, glo, 0, st) : exchange_to_grids<2>(p, dm.N, g, smem, h0, ghi, glo, 0, st);
    }
    if (e != cudaSuccess) return e;
    p->launches += 1;
    e = ffk_inverse_transform_tc(p, h0, g, out, st);
    if (e != cudaSuccess) return e;
    if (p->pipe_out) {                             // host-buffer entry point: hand this group of heads to the copy stream
      cudaEvent_t ev = p->ev_copy[FF_COPY_EVENTS + h0 / G];
      e = cudaEventRecord(ev, st);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(p->copy_stream, ev, 0);
      if (e == cudaSuccess)
        e = cudaMemcpyAsync((char*)p->pipe_out_host + (size_t)h0 * p->pipe_head_bytes, (const char*)out + (size_t)h0 * p->pipe_head_bytes,
                            (size_t)g * p->pipe_head_bytes, cudaMemcpyDeviceToHost, p->copy_stream);
      if (e != cudaSuccess) return e;
    }
  }
  return cudaSuccess;
}

template <typename ST>
static cudaError_t exchange_inverse_t(ff_plan* p, void* out, cudaStream_t st) {
  const FFDims& dm = p->dm;
  const int G = p->lay.group;
  DctPassParams P{};
  P.BH = dm.BH; P.N_d = dm.N * dm.d; P.dm = dm;
  const size_t smem = (size_t)3 * dm.m * dm.d * sizeof(float);
  for (int h0 = 0; h0 < dm.BH; h0 += G) {
    const int g = (dm.BH - h0 < G) ? dm.BH - h0 : G;
    const int rounds = exc_rounds(dm.N, g, p->sm_count);
    dim3 grid((unsigned)((dm.N + (long long)EXC_WARPS * rounds - 1) / ((long long)EXC_WARPS * rounds)), (unsigned)g);
    cudaError_t e = cudaSuccess;
#define FF_EXC(DPL)                                                                                                   \
  e = cudaFuncSetAttribute(exchange_recombine_kernel<ST, DPL, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
  if (e == cudaSuccess) exchange_recombine_kernel<ST, DPL, float><<<grid, EXC_WARPS * 32, smem, st>>>(p->buf, dm, h0, p->buf.scratchA, (float*)nullptr, 0, rounds);
    switch (dm.d / 32) {
      case 1: FF_EXC(1) break;
      case 2: FF_EXC(2) break;
      case 3: FF_EXC(3) break;
      default: FF_EXC(4) break;
    }
#undef FF_EXC
    if (e != cudaSuccess) return e;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    P.group_start = h0;
    // inverse along t, h, w with the transposed matrices
    P.src[0] = p->buf.scratchA; P.dst = p->buf.scratchB; P.mat = p->basis_t[0];
    P.n = dm.T; P.inner = dm.H * dm.W * dm.d; P.outer = 1;
    e = launch_dct_pass<ST, 1>(P, g, st);
    if (e != cudaSuccess) return e;
    P.src[0] = p->buf.scratchB; P.dst = p->buf.scratchA; P.mat = p->basis_t[1];
    P.n = dm.H; P.inner = dm.W * dm.d; P.outer = dm.T;
    e = launch_dct_pass<ST, 1>(P, g, st);
    if (e != cudaSuccess) return e;
    P.src[0] = p->buf.scratchA; P.dst = out; P.mat = p->basis_t[2];
    P.n = dm.W; P.inner = dm.d; P.outer = dm.T * dm.H;
    e = launch_dct_pass<ST, 3>(P, g, st);
    if (e != cudaSuccess) return e;
    p->launches += 4;
  }
  return cudaSuccess;
}

cudaError_t ffk_exchange_inverse(ff_plan* p, void* out, cudaStream_t st) {
  if (p->dct_tc_ok && !(p->attn_impl & 2)) return exchange_inverse_tc(p, out, st);
  return p->dm.fp32 ? exchange_inverse_t<float>(p, out, st) : exchange_inverse_t<__nv_bfloat16>(p, out, st);
}
