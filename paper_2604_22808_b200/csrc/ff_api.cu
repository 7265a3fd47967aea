// Host side of the C ABI: configuration checks, band arithmetic, workspace layout, plan lifetime
// and the launch sequence of the forward.  No device code lives here.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "ff_internal.h"

static thread_local char g_err[512] = "";

void ff_set_thread_error(const char* msg) { snprintf(g_err, 512, "%s", msg ? msg : ""); }

static ff_status_t fail(ff_plan* p, ff_status_t code, const char* fmt, const char* a = "", long long x = 0,
                        long long y = 0) {
  char* dst = p ? p->err : g_err;
  snprintf(dst, 512, fmt, a, x, y);
  return code;
}

#define FF_CUDA(p, call)                                                                        \
  do {                                                                                          \
    cudaError_t e__ = (call);                                                                   \
    if (e__ != cudaSuccess) return fail((p), FF_ERR_CUDA, "CUDA error: %s (" #call ")", cudaGetErrorString(e__)); \
  } while (0)

static void dims_from_cfg(const ff_config_t& c, FFDims* dm) {
  dm->B = c.batch; dm->T = c.T; dm->H = c.H; dm->W = c.W; dm->heads = c.heads; dm->d = c.head_dim;
  dm->BH = c.batch * c.heads;
  for (int a = 0; a < 3; ++a) { dm->L[a] = c.low_cut[a]; dm->M[a] = c.mid_cut[a]; }
  dm->r = c.low_compress; dm->b = c.mid_block; dm->s = c.mid_stride; dm->R = c.high_radius;
  dm->m = c.n_summary; dm->hid = c.router_hidden; dm->dt = c.t_embed_dim;
  dm->fp32 = (c.dtype == FF_FP32);
  dm->pattern = c.mid_pattern;
  dm->N = (long long)c.T * c.H * c.W;
  dm->Nlow = (long long)c.low_cut[0] * c.low_cut[1] * c.low_cut[2];
  dm->Nbar = (dm->Nlow + c.low_compress - 1) / (c.low_compress > 0 ? c.low_compress : 1);
  dm->Nmid = (long long)c.mid_cut[0] * c.mid_cut[1] * c.mid_cut[2] - dm->Nlow;
  dm->Nhigh = dm->N - (long long)c.mid_cut[0] * c.mid_cut[1] * c.mid_cut[2];
  dm->nb = (dm->Nmid + c.mid_block - 1) / (c.mid_block > 0 ? c.mid_block : 1);
}

extern "C" ff_status_t ff_config_validate(const ff_config_t* c) {
  if (!c) return fail(nullptr, FF_ERR_INVALID_ARG, "cfg is NULL%s");
  if (c->batch < 1 || c->T < 1 || c->H < 1 || c->W < 1 || c->heads < 1 || c->head_dim < 1)
    return fail(nullptr, FF_ERR_INVALID_ARG, "batch, grid, heads and head_dim must be positive%s");
  if (c->dtype != FF_BF16 && c->dtype != FF_FP32) return fail(nullptr, FF_ERR_INVALID_ARG, "dtype must be FF_BF16 or FF_FP32%s");
  const int n[3] = {c->T, c->H, c->W};
  for (int a = 0; a < 3; ++a) {
    if (c->low_cut[a] < 0 || c->low_cut[a] > c->mid_cut[a] || c->mid_cut[a] > n[a])
      return fail(nullptr, FF_ERR_INVALID_ARG, "cut-offs must satisfy 0 <= L_a <= M_a <= n_a (axis %s%lld)", "", a);
  }
  if (c->low_compress < 1 || c->mid_block < 1 || c->mid_stride < 1 || c->high_radius < 0 || c->n_summary < 0)
    return fail(nullptr, FF_ERR_INVALID_ARG, "need r >= 1, b >= 1, s >= 1, R >= 0, m >= 0%s");
  if (c->router_hidden < 1 || c->t_embed_dim < 2 || (c->t_embed_dim & 1))
    return fail(nullptr, FF_ERR_INVALID_ARG, "router_hidden >= 1 and an even t_embed_dim >= 2 are required%s");
  if (c->head_dim % 32 != 0 || c->head_dim > 128)
    return fail(nullptr, FF_ERR_UNSUPPORTED, "head_dim must be a multiple of 32 and <= 128%s");
  if (c->T > 128 || c->H > 128 || c->W > 128) return fail(nullptr, FF_ERR_UNSUPPORTED, "axis lengths above 128 are not supported%s");
  if (c->router_hidden > 1024 || c->n_summary > 64) return fail(nullptr, FF_ERR_UNSUPPORTED, "router_hidden <= 1024 and m <= 64 are supported%s");
  if (c->transform != FF_TRANSFORM_DCT && c->transform != FF_TRANSFORM_HAAR)
    return fail(nullptr, FF_ERR_INVALID_ARG, "transform must be FF_TRANSFORM_DCT or FF_TRANSFORM_HAAR%s");
  if (c->mid_pattern != FF_MID_STRIDED && c->mid_pattern != FF_MID_ANCHOR)
    return fail(nullptr, FF_ERR_INVALID_ARG, "mid_pattern must be FF_MID_STRIDED or FF_MID_ANCHOR%s");
  if (c->transform == FF_TRANSFORM_HAAR)
    for (int a = 0; a < 3; ++a)
      if (n[a] & (n[a] - 1)) return fail(nullptr, FF_ERR_UNSUPPORTED, "the Haar transform needs power-of-two axis lengths%s");
  FFDims dm; dims_from_cfg(*c, &dm);
  // Two bands ("Number of bands", L = 2): mid cut-offs equal to the low cut-offs leave the mid band empty, and
  // the layer runs with the low and the high band only.  The low and the high band must exist.
  if (dm.Nlow < 1 || dm.Nhigh < 1) return fail(nullptr, FF_ERR_EMPTY_BAND, "the cut-offs leave the low or the high band empty%s");
  return FF_OK;
}

extern "C" ff_status_t ff_band_sizes(const ff_config_t* c, int64_t sizes[4]) {
  if (!sizes) return fail(nullptr, FF_ERR_INVALID_ARG, "sizes is NULL%s");
  ff_status_t s = ff_config_validate(c);
  if (s != FF_OK && s != FF_ERR_EMPTY_BAND && s != FF_ERR_UNSUPPORTED) return s;
  FFDims dm; dims_from_cfg(*c, &dm);
  sizes[0] = dm.Nlow; sizes[1] = dm.Nbar; sizes[2] = dm.Nmid; sizes[3] = dm.Nhigh;
  return FF_OK;
}

extern "C" ff_status_t ff_band_rank(const ff_config_t* c, int32_t kt, int32_t kh, int32_t kw, int32_t* band,
                                    int64_t* rank) {
  if (!band || !rank) return fail(nullptr, FF_ERR_INVALID_ARG, "band/rank is NULL%s");
  ff_status_t s = ff_config_validate(c);
  if (s != FF_OK && s != FF_ERR_EMPTY_BAND && s != FF_ERR_UNSUPPORTED) return s;
  if (kt < 0 || kh < 0 || kw < 0 || kt >= c->T || kh >= c->H || kw >= c->W)
    return fail(nullptr, FF_ERR_INVALID_ARG, "coefficient index outside the grid%s");
  FFDims dm; dims_from_cfg(*c, &dm);
  long long rk;
  *band = ff_band_rank_of(dm, kt, kh, kw, &rk);
  *rank = rk;
  return FF_OK;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

void ff_compute_layout(const FFDims& dm, bool with_staging, FFLayout* lay) {
  const size_t e = dm.fp32 ? 4 : 2;
  const size_t d = dm.d, BH = dm.BH;
  // Tensor-heads per generic transform launch: as many as fit two fp32 scratch grids of ~1 GiB each.
  const size_t per = (size_t)dm.N * d * 4;
  size_t G = ((size_t)1 << 30) / per;
  if (G < 1) G = 1;
  if (G > 3 * BH) G = 3 * BH;
  lay->group = (int)G;
  // Tensor-core transform: as many tensor-heads per launch as fit ~8 GiB of scratch (at least 3): every launch
  // pays a ramp-up and a tail, and fewer, longer launches measured faster (64K tokens, 72 tensor-heads: one group against
  // 32 + 32 + 8, 1.58 against 1.66 ms for the forward transform).  The host-buffer entry point
  // works in groups of a quarter of that, so that the transform of one group overlaps the copy of the next.
  size_t Gt = ((size_t)8 << 30) / (4 * (size_t)dm.N * d * 2);
  if (Gt < 3) Gt = 3;
  if (Gt > 3 * BH) Gt = 3 * BH;
  lay->tc_group = (int)Gt;
  size_t Gp = ((size_t)2 << 30) / (4 * (size_t)dm.N * d * 2);
  if (Gp < 3) Gp = 3;
  if (Gp > Gt) Gp = Gt;
  lay->tc_group_pipe = (int)Gp;
  const size_t tc_scratch = ffk_dct_tc_supported(dm) ? ffk_dct_tc_scratch_bytes(dm, (int)Gt) : 0;
  const size_t sizes[21] = {
      3 * BH * (size_t)dm.Nlow * d * 4,   // 0 spec_low
      3 * BH * (size_t)dm.Nmid * d * e,   // 1 spec_mid
      3 * BH * (size_t)dm.Nhigh * d * e,  // 2 spec_high
      3 * BH * (size_t)dm.Nbar * d * 4,   // 3 pooled
      BH * (size_t)dm.Nbar * d * 4,       // 4 y_low
      BH * (size_t)dm.Nmid * d * e,       // 5 y_mid
      BH * (size_t)dm.Nhigh * d * e,      // 6 y_high
      BH * 3 * (size_t)(dm.m > 0 ? dm.m : 1) * d * 4,  // 7 summary
      (size_t)dm.B * 3 * d * 8,           // 8 energy
      BH,                                 // 9 alloc
      (size_t)dm.B * 3 * 4,               // 10 pi
      (size_t)dm.B * 4,                   // 11 timestep
      256,                                // 12 status
      tc_scratch > 2 * G * per ? tc_scratch - G * per : G * per,   // 13 scratchA (the tensor-core transform
      G * per,                            // 14 scratchB                  uses A and B as one region)
      with_staging ? BH * (size_t)dm.N * d * e : 0,  // 15..18 staging
      with_staging ? BH * (size_t)dm.N * d * e : 0,
      with_staging ? BH * (size_t)dm.N * d * e : 0,
      with_staging ? BH * (size_t)dm.N * d * e : 0,
      ffk_tc_work_bytes(),                // 19 worklist
      dm.fp32 ? 0 : 3 * BH * (size_t)dm.Nbar * d * 2,   // 20 pooled low band as bf16
  };
  size_t off = 0;
  for (int i = 0; i < 21; ++i) { lay->off[i] = off; off += align_up(sizes[i], 256); }
  lay->total = off;
}

extern "C" ff_status_t ff_workspace_bytes(const ff_config_t* c, size_t* bytes) {
  if (!bytes) return fail(nullptr, FF_ERR_INVALID_ARG, "bytes is NULL%s");
  ff_status_t s = ff_config_validate(c);
  if (s != FF_OK) return s;
  FFDims dm; dims_from_cfg(*c, &dm);
  FFLayout lay; ff_compute_layout(dm, false, &lay);
  *bytes = lay.total;
  return FF_OK;
}

extern "C" ff_status_t ff_workspace_bytes_host(const ff_config_t* c, size_t* bytes) {
  if (!bytes) return fail(nullptr, FF_ERR_INVALID_ARG, "bytes is NULL%s");
  ff_status_t s = ff_config_validate(c);
  if (s != FF_OK) return s;
  FFDims dm; dims_from_cfg(*c, &dm);
  FFLayout lay; ff_compute_layout(dm, true, &lay);
  *bytes = lay.total;
  return FF_OK;
}

static ff_status_t upload(ff_plan* p, float** dst, const float* src, size_t n) {
  FF_CUDA(p, cudaMalloc((void**)dst, n * sizeof(float)));
  FF_CUDA(p, cudaMemcpy(*dst, src, n * sizeof(float), cudaMemcpyHostToDevice));
  return FF_OK;
}

extern "C" ff_status_t ff_destroy(ff_plan_t* p) {
  if (!p) return FF_OK;
  for (int a = 0; a < 3; ++a) { cudaFree(p->basis[a]); cudaFree(p->basis_t[a]); }
  if (p->ev[0]) for (int i = 0; i <= FF_STAGE_COUNT; ++i) cudaEventDestroy(p->ev[i]);
  if (p->copy_stream) {
    for (int i = 0; i <= 2 * FF_COPY_EVENTS; ++i) cudaEventDestroy(p->ev_copy[i]);
    cudaStreamDestroy(p->copy_stream);
  }
  cudaFree(p->dct2_images); cudaFree(p->pos_table);
  cudaFree(p->W1); cudaFree(p->b1); cudaFree(p->W2); cudaFree(p->b2); cudaFree(p->U);
  delete p;
  return FF_OK;
}

extern "C" ff_status_t ff_plan_create(const ff_config_t* c, const ff_weights_t* w, ff_plan_t** out) {
  if (!out) return fail(nullptr, FF_ERR_INVALID_ARG, "out_plan is NULL%s");
  *out = nullptr;
  ff_status_t s = ff_config_validate(c);
  if (s != FF_OK) return s;
  ff_plan* p = new (std::nothrow) ff_plan();
  if (!p) return fail(nullptr, FF_ERR_INVALID_ARG, "out of host memory%s");
  memset(p, 0, sizeof(*p));
  p->cfg = *c;
  dims_from_cfg(*c, &p->dm);
  cudaError_t ce = cudaGetDevice(&p->device);
  if (ce == cudaSuccess) ce = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device);
  if (ce != cudaSuccess) {
    fail(nullptr, FF_ERR_CUDA, "no usable CUDA device: %s", cudaGetErrorString(ce));
    delete p;
    return FF_ERR_CUDA;
  }
  // The 1-D transform matrices C[k][i], evaluated in double: DCT-II, alpha_k cos(pi (2i+1) k / (2n)), or the
  // orthonormal Haar wavelets (row 0 constant; row 2^j + q is +-sqrt(2^j / n) on the halves of the q-th block of
  // n / 2^j positions), rows from the coarsest scale to the finest.
  const int n[3] = {c->T, c->H, c->W};
  for (int a = 0; a < 3 && s == FF_OK; ++a) {
    std::vector<float> C((size_t)n[a] * n[a]), Ct((size_t)n[a] * n[a]);
    for (int k = 0; k < n[a]; ++k)
      for (int i = 0; i < n[a]; ++i) {
        double v;
        if (c->transform == FF_TRANSFORM_HAAR) {
          if (k == 0) v = sqrt(1.0 / n[a]);
          else {
            int j = 0;
            while ((2 << j) <= k) ++j;                       // level: 2^j <= k < 2^(j+1)
            const int q = k - (1 << j), block = n[a] >> j;
            const double amp = sqrt((double)(1 << j) / n[a]);
            v = (i < q * block || i >= (q + 1) * block) ? 0.0 : (i < q * block + block / 2 ? amp : -amp);
          }
        } else {
          const double alpha = (k == 0) ? sqrt(1.0 / n[a]) : sqrt(2.0 / n[a]);
          v = alpha * cos(M_PI * (2.0 * i + 1.0) * k / (2.0 * n[a]));
        }
        C[(size_t)k * n[a] + i] = (float)v;
        Ct[(size_t)i * n[a] + k] = (float)v;
      }
    s = upload(p, &p->basis[a], C.data(), C.size());
    if (s == FF_OK) s = upload(p, &p->basis_t[a], Ct.data(), Ct.size());
    if (s == FF_OK && ffk_dct_tc_supported(p->dm) &&
        !(ffk_dct2_build_image(p, a, 0, C.data(), n[a]) && ffk_dct2_build_image(p, a, 1, Ct.data(), n[a])))
      s = fail(p, FF_ERR_CUDA, "could not upload the transform matrix images%s");
  }
  p->dct2_ok = s == FF_OK && p->dct2_images && ffk_dct2_supported(p->dm, &p->dct2_axis2, nullptr);
  const size_t d = c->head_dim, hid = c->router_hidden, nin = 3 * d + c->t_embed_dim;
  if (s == FF_OK && w && w->W1 && w->b1 && w->W2 && w->b2) {
    s = upload(p, &p->W1, w->W1, hid * nin);
    if (s == FF_OK) s = upload(p, &p->b1, w->b1, hid);
    if (s == FF_OK) s = upload(p, &p->W2, w->W2, 3 * hid);
    if (s == FF_OK) s = upload(p, &p->b2, w->b2, 3);
    p->has_router = true;
  }
  if (s == FF_OK) {
    std::vector<float> U(3 * d * d, 0.f);
    p->identity_u = !(w && w->U);
    if (w && w->U) memcpy(U.data(), w->U, U.size() * sizeof(float));
    else for (size_t l = 0; l < 3; ++l) for (size_t i = 0; i < d; ++i) U[(l * d + i) * d + i] = 1.f;
    s = upload(p, &p->U, U.data(), U.size());
  }
  if (s == FF_OK && ffk_exchange_tc_supported(p->dm) && !ffk_exchange_tc_build_tables(p))
    s = fail(p, FF_ERR_CUDA, "could not upload the band position tables%s");
  if (s != FF_OK) {
    snprintf(g_err, 512, "%s", p->err);
    ff_destroy(p);
    return s;
  }
  ff_compute_layout(p->dm, false, &p->lay);
  *out = p;
  return FF_OK;
}

extern "C" ff_status_t ff_plan_workspace_bytes(const ff_plan_t* p, size_t* bytes) {
  if (!p || !bytes) return fail(nullptr, FF_ERR_INVALID_ARG, "plan or bytes is NULL%s");
  *bytes = p->lay.total;
  return FF_OK;
}

extern "C" ff_status_t ff_band_info(const ff_plan_t* p, int64_t sizes[4]) {
  if (!p || !sizes) return fail(nullptr, FF_ERR_INVALID_ARG, "plan or sizes is NULL%s");
  sizes[0] = p->dm.Nlow; sizes[1] = p->dm.Nbar; sizes[2] = p->dm.Nmid; sizes[3] = p->dm.Nhigh;
  return FF_OK;
}

extern "C" ff_status_t ff_plan_set_workspace(ff_plan_t* p, void* ptr, size_t bytes) {
  if (!p) return fail(nullptr, FF_ERR_INVALID_ARG, "plan is NULL%s");
  if (!ptr) return fail(p, FF_ERR_WORKSPACE, "workspace pointer is NULL%s");
  if (((uintptr_t)ptr) & 255) return fail(p, FF_ERR_WORKSPACE, "workspace must be 256-byte aligned%s");
  FFLayout plain, staged;
  ff_compute_layout(p->dm, false, &plain);
  ff_compute_layout(p->dm, true, &staged);
  if (bytes < plain.total)
    return fail(p, FF_ERR_WORKSPACE, "workspace too small%s: %lld bytes given, %lld needed", "", (long long)bytes, (long long)plain.total);
  p->ws_has_staging = bytes >= staged.total;
  p->lay = p->ws_has_staging ? staged : plain;
  p->ws = ptr; p->ws_bytes = bytes;
  char* base = (char*)ptr;
  const size_t* o = p->lay.off;
  FFBuffers& b = p->buf;
  b.spec_low = (float*)(base + o[0]); b.spec_mid = base + o[1]; b.spec_high = base + o[2];
  b.pooled = (float*)(base + o[3]); b.y_low = (float*)(base + o[4]); b.y_mid = base + o[5]; b.y_high = base + o[6];
  b.summary = (float*)(base + o[7]); b.energy = (double*)(base + o[8]); b.alloc = (uint8_t*)(base + o[9]);
  b.pi = (float*)(base + o[10]); b.timestep = (float*)(base + o[11]); b.status = (int*)(base + o[12]);
  b.scratchA = (float*)(base + o[13]); b.scratchB = (float*)(base + o[14]);
  b.stage_q = p->ws_has_staging ? base + o[15] : nullptr; b.stage_k = p->ws_has_staging ? base + o[16] : nullptr;
  b.stage_v = p->ws_has_staging ? base + o[17] : nullptr; b.stage_out = p->ws_has_staging ? base + o[18] : nullptr;
  b.work = (int*)(base + o[19]);
  b.pooled_bf = p->dm.fp32 ? nullptr : (__nv_bfloat16*)(base + o[20]);
  FF_CUDA(p, cudaMemset(b.status, 0, 256));
  p->tc_ok = ffk_tc_supported(p->dm) && ffk_tc_prepare(p);
  p->xtc_ok = p->pos_table && ffk_exchange_tc_supported(p->dm) && ffk_exchange_tc_prepare(p);
  // The tensor-core transform shares the scratch region (scratchA and scratchB are adjacent).
  p->dct_tc_ok = false;
  if (ffk_dct_tc_supported(p->dm)) {
    const size_t room = (size_t)((char*)base + o[14] - (char*)b.scratchA) + (size_t)p->lay.group * p->dm.N * p->dm.d * 4;
    const int G = p->lay.tc_group;
    if (p->dct2_images && ffk_dct_tc_scratch_bytes(p->dm, G) <= room) { p->dct_tc_ok = true; p->dct_group = G; }
  }
  return FF_OK;
}

extern "C" const char* ff_last_error(const ff_plan_t* p) { return p ? p->err : g_err; }

extern "C" ff_status_t ff_plan_set_attention_impl(ff_plan_t* p, int32_t impl) {
  if (!p) return fail(nullptr, FF_ERR_INVALID_ARG, "plan is NULL%s");
  if (impl < 0 || impl > 7) return fail(p, FF_ERR_INVALID_ARG, "impl must be in [0, 7]%s");
  p->attn_impl = impl;
  return FF_OK;
}

extern "C" ff_status_t ff_plan_kernel_info(const ff_plan_t* p, int32_t info[4]) {
  if (!p || !info) return fail(nullptr, FF_ERR_INVALID_ARG, "plan or info is NULL%s");
  int cs = 0;
  const bool fused = p->dct_tc_ok && p->dct2_ok && !(p->attn_impl & 6) && ffk_dct2_supported(p->dm, nullptr, &cs);
  info[0] = fused ? 1 : 0; info[1] = fused ? cs : 0;
  info[2] = (p->tc_ok && !(p->attn_impl & 1)) ? 1 : 0; info[3] = (info[2] && p->low_tc_ok) ? 1 : 0;
  return FF_OK;
}

extern "C" ff_status_t ff_plan_last_launches(const ff_plan_t* p, int64_t* n) {
  if (!p || !n) return fail(nullptr, FF_ERR_INVALID_ARG, "plan or output is NULL%s");
  *n = p->launches;
  return FF_OK;
}

extern "C" ff_status_t ff_plan_device_status(ff_plan_t* p, void* stream) {
  if (!p) return fail(nullptr, FF_ERR_INVALID_ARG, "plan is NULL%s");
  if (!p->ws) return fail(p, FF_ERR_WORKSPACE, "no workspace set%s");
  cudaStream_t st = (cudaStream_t)stream;
  int word = 0;
  FF_CUDA(p, cudaMemcpyAsync(&word, p->buf.status, sizeof(int), cudaMemcpyDeviceToHost, st));
  FF_CUDA(p, cudaStreamSynchronize(st));
  if (word != 0) {
    FF_CUDA(p, cudaMemsetAsync(p->buf.status, 0, sizeof(int), st));
    return fail(p, (ff_status_t)(word & 0xff), "device status word reports an error%s (status %lld, kernel %lld)", "", word & 0xff, word >> 8);
  }
  return FF_OK;
}

static ff_status_t check_call(ff_plan* p, const void* Q, const void* K, const void* V) {
  if (!p) return fail(nullptr, FF_ERR_INVALID_ARG, "plan is NULL%s");
  if (!Q || !K || !V) return fail(p, FF_ERR_INVALID_ARG, "Q, K or V is NULL%s");
  if (!p->ws) return fail(p, FF_ERR_WORKSPACE, "ff_plan_set_workspace has not been called%s");
  if ((((uintptr_t)Q) | ((uintptr_t)K) | ((uintptr_t)V)) & 15)
    return fail(p, FF_ERR_INVALID_ARG, "Q, K and V must be 16-byte aligned%s");
  return FF_OK;
}

extern "C" ff_status_t ff_plan_set_profiling(ff_plan_t* p, int32_t enable) {
  if (!p) return fail(nullptr, FF_ERR_INVALID_ARG, "plan is NULL%s");
  if (enable && !p->ev[0])
    for (int i = 0; i <= FF_STAGE_COUNT; ++i) FF_CUDA(p, cudaEventCreate(&p->ev[i]));
  p->profiling = enable != 0;
  return FF_OK;
}

extern "C" ff_status_t ff_plan_stage_times(ff_plan_t* p, float ms[FF_STAGE_COUNT], int64_t launches[FF_STAGE_COUNT]) {
  if (!p || !ms || !launches) return fail(nullptr, FF_ERR_INVALID_ARG, "plan or output is NULL%s");
  if (!p->profiling) return fail(p, FF_ERR_INVALID_ARG, "profiling is not enabled%s");
  FF_CUDA(p, cudaEventSynchronize(p->ev[FF_STAGE_COUNT]));
  for (int i = 0; i < FF_STAGE_COUNT; ++i) {
    FF_CUDA(p, cudaEventElapsedTime(&ms[i], p->ev[i], p->ev[i + 1]));
    launches[i] = p->stage_launches[i];
  }
  return FF_OK;
}

// Stage boundary: remembers the launches of the stage that just ended and records its end event.
static cudaError_t mark(ff_plan* p, int boundary, cudaStream_t st) {
  static thread_local long long before = 0;
  if (boundary == 0) before = 0;
  else { p->stage_launches[boundary - 1] = p->launches - before; before = p->launches; }
  return p->profiling ? cudaEventRecord(p->ev[boundary], st) : cudaSuccess;
}

// Transform, statistics and router: the part ff_route and an internally routed ff_forward share.
static ff_status_t transform_and_route(ff_plan* p, const void* Q, const void* K, const void* V, const float* timestep,
                                       bool route, cudaStream_t st) {
  FF_CUDA(p, mark(p, 0, st));
  if (route) {
    if (!p->has_router) return fail(p, FF_ERR_NOT_ROUTED, "the plan was created without router weights%s");
    if (!timestep) return fail(p, FF_ERR_NOT_ROUTED, "neither an allocation nor a timestep was given%s");
    FF_CUDA(p, cudaMemcpyAsync(p->buf.timestep, timestep, sizeof(float) * p->dm.B, cudaMemcpyHostToDevice, st));
    FF_CUDA(p, cudaMemsetAsync(p->buf.energy, 0, sizeof(double) * p->dm.B * 3 * p->dm.d, st));
  }
  const bool tc_transform = p->dct_tc_ok && !(p->attn_impl & 2);
  if (tc_transform) FF_CUDA(p, ffk_forward_transform_tc(p, Q, K, V, route, st));   // band energies come from its epilogue
  else FF_CUDA(p, ffk_forward_transform(p, Q, K, V, st));
  FF_CUDA(p, mark(p, 1, st));
  if (route) {
    if (!tc_transform) FF_CUDA(p, ffk_band_energy(p, st));
    FF_CUDA(p, ffk_router(p, p->buf.alloc, st));
  }
  FF_CUDA(p, mark(p, 2, st));
  return FF_OK;
}

extern "C" ff_status_t ff_route(ff_plan_t* p, const void* Q, const void* K, const void* V, const float* timestep,
                                uint8_t* alloc_dev, uint8_t* alloc_host, float* pi_host, void* stream) {
  ff_status_t s = check_call(p, Q, K, V);
  if (s != FF_OK) return s;
  if (!timestep) return fail(p, FF_ERR_INVALID_ARG, "timestep is NULL%s");
  cudaStream_t st = (cudaStream_t)stream;
  p->launches = 0;
  s = transform_and_route(p, Q, K, V, timestep, true, st);
  if (s != FF_OK) return s;
  if (alloc_dev) FF_CUDA(p, cudaMemcpyAsync(alloc_dev, p->buf.alloc, p->dm.BH, cudaMemcpyDeviceToDevice, st));
  if (alloc_host) FF_CUDA(p, cudaMemcpyAsync(alloc_host, p->buf.alloc, p->dm.BH, cudaMemcpyDeviceToHost, st));
  if (pi_host) FF_CUDA(p, cudaMemcpyAsync(pi_host, p->buf.pi, sizeof(float) * 3 * p->dm.B, cudaMemcpyDeviceToHost, st));
  if (alloc_host || pi_host) FF_CUDA(p, cudaStreamSynchronize(st));
  return FF_OK;
}

extern "C" ff_status_t ff_forward(ff_plan_t* p, const void* Q, const void* K, const void* V, const uint8_t* alloc_dev,
                                  const float* timestep, void* out, void* stream) {
  ff_status_t s = check_call(p, Q, K, V);
  if (s != FF_OK) return s;
  if (!out) return fail(p, FF_ERR_INVALID_ARG, "out is NULL%s");
  if (((uintptr_t)out) & 15) return fail(p, FF_ERR_INVALID_ARG, "out must be 16-byte aligned%s");
  if (!alloc_dev && !timestep) return fail(p, FF_ERR_NOT_ROUTED, "neither an allocation nor a timestep was given%s");
  cudaStream_t st = (cudaStream_t)stream;
  p->launches = 0;
  s = transform_and_route(p, Q, K, V, timestep, alloc_dev == nullptr, st);
  if (s != FF_OK) return s;
  if (alloc_dev) FF_CUDA(p, cudaMemcpyAsync(p->buf.alloc, alloc_dev, p->dm.BH, cudaMemcpyDeviceToDevice, st));
  FF_CUDA(p, ffk_pool_low(p, st));
  if (p->tc_ok && !(p->attn_impl & 1)) {
    // the tensor-core launch takes the high band, the strided mid band and a long pooled low band
    const int simt_bands = (p->low_tc_ok ? 0 : FF_BAND_LOW) | (p->dm.pattern == FF_MID_ANCHOR ? FF_BAND_MID : 0);
    if (simt_bands) FF_CUDA(p, ffk_attention_simt(p, simt_bands, st));
    FF_CUDA(p, ffk_attention_tc(p, st));
  } else {
    FF_CUDA(p, ffk_attention_simt(p, FF_BAND_LOW | FF_BAND_MID | FF_BAND_HIGH, st));
  }
  FF_CUDA(p, mark(p, 3, st));
  if (p->dm.m > 0) FF_CUDA(p, ffk_summaries(p, st));
  FF_CUDA(p, mark(p, 4, st));
  FF_CUDA(p, ffk_exchange_inverse(p, out, st));
  FF_CUDA(p, mark(p, 5, st));
  return FF_OK;
}

extern "C" ff_status_t ff_forward_projected(ff_plan_t* p, const void* X, const void* Wqkv, const void* Wo,
                                            const uint8_t* alloc_dev, const float* timestep, void* out, void* stream) {
  if (!p) return fail(nullptr, FF_ERR_INVALID_ARG, "plan is NULL%s");
  if (!X || !Wqkv || !Wo || !out) return fail(p, FF_ERR_INVALID_ARG, "X, Wqkv, Wo or out is NULL%s");
  if ((((uintptr_t)X) | ((uintptr_t)Wqkv) | ((uintptr_t)Wo) | ((uintptr_t)out)) & 15)
    return fail(p, FF_ERR_INVALID_ARG, "X, Wqkv, Wo and out must be 16-byte aligned%s");
  if (!p->ws) return fail(p, FF_ERR_WORKSPACE, "ff_plan_set_workspace has not been called%s");
  if (!p->ws_has_staging) return fail(p, FF_ERR_WORKSPACE, "workspace lacks staging space: size it with ff_workspace_bytes_host%s");
  if (!ffk_proj_supported(p->dm))
    return fail(p, FF_ERR_UNSUPPORTED, "projections need bf16, head_dim 64 or 128, tokens %% 128 == 0 and heads * head_dim %% 256 == 0%s");
  if (!alloc_dev && !timestep) return fail(p, FF_ERR_NOT_ROUTED, "neither an allocation nor a timestep was given%s");
  cudaStream_t st = (cudaStream_t)stream;
  FF_CUDA(p, ffk_project_qkv(p, X, Wqkv, p->buf.stage_q, p->buf.stage_k, p->buf.stage_v, st));
  ff_status_t s = ff_forward(p, p->buf.stage_q, p->buf.stage_k, p->buf.stage_v, alloc_dev, timestep, p->buf.stage_out, st);
  if (s != FF_OK) return s;
  FF_CUDA(p, ffk_project_out(p, p->buf.stage_out, Wo, out, st));
  p->launches += 1;                                 // (ff_forward restarted the count: add the first projection)
  return FF_OK;
}

extern "C" ff_status_t ff_forward_host(ff_plan_t* p, const void* Qh, const void* Kh, const void* Vh,
                                       const uint8_t* alloc_host, const float* timestep, void* out_host, void* stream) {
  if (!p) return fail(nullptr, FF_ERR_INVALID_ARG, "plan is NULL%s");
  if (!Qh || !Kh || !Vh || !out_host) return fail(p, FF_ERR_INVALID_ARG, "a host buffer is NULL%s");
  if (!p->ws) return fail(p, FF_ERR_WORKSPACE, "ff_plan_set_workspace has not been called%s");
  if (!p->ws_has_staging) return fail(p, FF_ERR_WORKSPACE, "workspace lacks staging space: size it with ff_workspace_bytes_host%s");
  cudaStream_t st = (cudaStream_t)stream;
  const FFDims& dm = p->dm;
  const size_t head_bytes = (size_t)dm.N * dm.d * (dm.fp32 ? 4 : 2);
  const size_t bytes = (size_t)dm.BH * head_bytes;
  // On the tensor-core path the copies are pipelined with the transforms: the forward transform works
  // through Q, K, V in groups of tensor-heads and waits only for its own group's copy; the inverse
  // hands every finished group of heads to the copy stream.
  // (smaller groups for this call: see ff_compute_layout; put back on every way out)
  struct GroupGuard {
    ff_plan* p; int saved;
    GroupGuard(ff_plan* q) : p(q), saved(q->dct_group) { if (q->lay.tc_group_pipe < q->dct_group) q->dct_group = q->lay.tc_group_pipe; }
    ~GroupGuard() { p->dct_group = saved; }
  } group_guard(p);
  const int G = p->dct_group;
  const int total = 3 * dm.BH;
  const bool piped = p->dct_tc_ok && !(p->attn_impl & 2) && G > 0 && (total + G - 1) / G <= FF_COPY_EVENTS &&
                     (dm.BH + G - 1) / G <= FF_COPY_EVENTS;
  if (piped && !p->copy_stream) {
    FF_CUDA(p, cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking));
    for (int i = 0; i <= 2 * FF_COPY_EVENTS; ++i) FF_CUDA(p, cudaEventCreateWithFlags(&p->ev_copy[i], cudaEventDisableTiming));
  }
  // The caller's masks travel through the tail of the (not yet used) output staging area.
  uint8_t* alloc_dev = nullptr;
  if (alloc_host) {
    alloc_dev = (uint8_t*)p->buf.stage_out;
    FF_CUDA(p, cudaMemcpyAsync(alloc_dev, alloc_host, dm.BH, cudaMemcpyHostToDevice, st));
  }
  if (piped) {
    // the copy stream starts after everything already queued on the caller's stream
    FF_CUDA(p, cudaEventRecord(p->ev_copy[2 * FF_COPY_EVENTS], st));
    FF_CUDA(p, cudaStreamWaitEvent(p->copy_stream, p->ev_copy[2 * FF_COPY_EVENTS], 0));
    const void* src[3] = {Qh, Kh, Vh};
    void* dst[3] = {p->buf.stage_q, p->buf.stage_k, p->buf.stage_v};
    for (int g0 = 0, gi = 0; g0 < total; g0 += G, ++gi) {
      const int g1 = g0 + G < total ? g0 + G : total;
      for (int th = g0; th < g1;) {                 // a group may straddle two tensors
        const int tensor = th / dm.BH, h = th % dm.BH;
        const int n = (g1 - th) < (dm.BH - h) ? (g1 - th) : (dm.BH - h);
        FF_CUDA(p, cudaMemcpyAsync((char*)dst[tensor] + (size_t)h * head_bytes, (const char*)src[tensor] + (size_t)h * head_bytes,
                                   (size_t)n * head_bytes, cudaMemcpyHostToDevice, p->copy_stream));
        th += n;
      }
      FF_CUDA(p, cudaEventRecord(p->ev_copy[gi], p->copy_stream));
    }
    p->pipe_in = p->pipe_out = true;
    p->pipe_out_host = out_host;
    p->pipe_head_bytes = head_bytes;
  } else {
    FF_CUDA(p, cudaMemcpyAsync(p->buf.stage_q, Qh, bytes, cudaMemcpyHostToDevice, st));
    FF_CUDA(p, cudaMemcpyAsync(p->buf.stage_k, Kh, bytes, cudaMemcpyHostToDevice, st));
    FF_CUDA(p, cudaMemcpyAsync(p->buf.stage_v, Vh, bytes, cudaMemcpyHostToDevice, st));
  }
  ff_status_t s = ff_forward(p, p->buf.stage_q, p->buf.stage_k, p->buf.stage_v, alloc_dev, timestep, p->buf.stage_out, st);
  const bool was_piped = p->pipe_out;
  p->pipe_in = p->pipe_out = false;
  if (s != FF_OK) { if (was_piped) cudaStreamSynchronize(p->copy_stream); return s; }
  if (was_piped) {
    FF_CUDA(p, cudaStreamSynchronize(p->copy_stream));
  } else {
    FF_CUDA(p, cudaMemcpyAsync(out_host, p->buf.stage_out, bytes, cudaMemcpyDeviceToHost, st));
  }
  FF_CUDA(p, cudaStreamSynchronize(st));
  return FF_OK;
}

extern "C" ff_status_t ff_get_tap(const ff_plan_t* p, int32_t which, const void** ptr, size_t* bytes) {
  if (!p || !ptr || !bytes) return fail(nullptr, FF_ERR_INVALID_ARG, "plan, dev_ptr or bytes is NULL%s");
  if (!p->ws) return FF_ERR_WORKSPACE;
  const FFDims& dm = p->dm;
  const size_t e = dm.fp32 ? 4 : 2, d = dm.d, BH = dm.BH;
  const FFBuffers& b = p->buf;
  switch (which) {
    case FF_TAP_SPEC_LOW: *ptr = b.spec_low; *bytes = 3 * BH * dm.Nlow * d * 4; break;
    case FF_TAP_SPEC_MID: *ptr = b.spec_mid; *bytes = 3 * BH * dm.Nmid * d * e; break;
    case FF_TAP_SPEC_HIGH: *ptr = b.spec_high; *bytes = 3 * BH * dm.Nhigh * d * e; break;
    case FF_TAP_POOLED_LOW: *ptr = b.pooled; *bytes = 3 * BH * dm.Nbar * d * 4; break;
    case FF_TAP_Y_LOW: *ptr = b.y_low; *bytes = BH * dm.Nbar * d * 4; break;
    case FF_TAP_Y_MID: *ptr = b.y_mid; *bytes = BH * dm.Nmid * d * e; break;
    case FF_TAP_Y_HIGH: *ptr = b.y_high; *bytes = BH * dm.Nhigh * d * e; break;
    case FF_TAP_SUMMARY: *ptr = b.summary; *bytes = BH * 3 * (size_t)dm.m * d * 4; break;
    case FF_TAP_ENERGY: *ptr = b.energy; *bytes = (size_t)dm.B * 3 * d * 8; break;
    case FF_TAP_ALLOC: *ptr = b.alloc; *bytes = BH; break;
    case FF_TAP_PI: *ptr = b.pi; *bytes = (size_t)dm.B * 3 * 4; break;
    default: return FF_ERR_INVALID_ARG;
  }
  return FF_OK;
}

// ------------------------------------------------------------------------------------------------
// Self-test of the bounded device-side wait every tensor-core kernel is built on: one CTA waits,
// with a limit of `limit_cycles`, on a barrier nobody ever arrives at; when the limit runs out the
// first waiter raises the CTA's abort flag, the second waiter (another warp) sees the flag and
// leaves too, and the CTA records FF_ERR_TIMEOUT in the plan's status word and returns.  Nothing
// hangs: the longest possible wait is the limit (at most 2e9 cycles, about a second).
// ------------------------------------------------------------------------------------------------
#include "ff_sm100.cuh"

namespace {
__global__ void bounded_wait_selftest_kernel(int* status, long long limit_cycles, int* observed) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) { sm100::mbar_init(&bar, 1); abort_flag = 0; sm100::fence_mbar_init(); }
  __syncthreads();
  bool ok = true;
  if (threadIdx.x == 0) ok = sm100::mbar_wait(&bar, 0, &abort_flag, limit_cycles);         // runs out
  if (threadIdx.x == 32) ok = sm100::mbar_wait(&bar, 0, &abort_flag, 4 * limit_cycles);    // leaves on the flag
  if (threadIdx.x == 0 || threadIdx.x == 32) atomicAdd(observed, ok ? 0 : 1);
  __syncthreads();
  if (threadIdx.x == 0 && abort_flag) atomicExch(status, FF_ERR_TIMEOUT | 0x500);
}
}  // namespace

extern "C" ff_status_t ff_plan_selftest_bounded_wait(ff_plan_t* p, int64_t limit_cycles, int32_t* waiters_released,
                                                     void* stream) {
  if (!p || !waiters_released) return fail(p, FF_ERR_INVALID_ARG, "plan or waiters_released is NULL%s");
  if (!p->ws) return fail(p, FF_ERR_WORKSPACE, "ff_plan_set_workspace has not been called%s");
  if (limit_cycles < 1 || limit_cycles > 2000000000LL) return fail(p, FF_ERR_INVALID_ARG, "limit_cycles must be in [1, 2e9]%s");
  cudaStream_t st = (cudaStream_t)stream;
  int* observed = p->buf.status + 1;               // the status region is 256 bytes; word 0 is the status
  FF_CUDA(p, cudaMemsetAsync(observed, 0, sizeof(int), st));
  bounded_wait_selftest_kernel<<<1, 64, 0, st>>>(p->buf.status, limit_cycles, observed);
  FF_CUDA(p, cudaGetLastError());
  FF_CUDA(p, cudaMemcpyAsync(waiters_released, observed, sizeof(int), cudaMemcpyDeviceToHost, st));
  FF_CUDA(p, cudaStreamSynchronize(st));
  return FF_OK;
}
