// Exported entry points that dispatch to the kernels: dense convolution forward, the unmerged
// inverted-residual block, workspace status, and the host-buffer entry point of the whole path.
#include <vector>

#include "common.cuh"

extern "C" const char *dc_status_string(dc_status s) {
  switch (s) {
    case DC_OK: return "ok";
    case DC_ERR_INVALID_ARG: return "invalid argument";
    case DC_ERR_SHAPE: return "shapes do not connect";
    case DC_ERR_UNSUPPORTED: return "unsupported configuration";
    case DC_ERR_NOT_MERGEABLE: return "skip group cannot be folded into one convolution";
    case DC_ERR_WORKSPACE: return "workspace missing or too small";
    case DC_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case DC_ERR_CUDA: return "CUDA call failed";
    case DC_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

extern "C" size_t dc_conv_workspace_bytes(void) { return sizeof(DcWsHeader); }

extern "C" const char *dc_conv_kernel_name(int n, int h, int w, const dc_geom *g, dc_dtype dtype) {
  if (dc_validate_geom(g) != DC_OK || g->groups != 1 || n <= 0 || h <= 0 || w <= 0) return nullptr;
  if (dtype == DC_F32) return "k_conv_dense_f32";
  if (dtype != DC_BF16) return nullptr;
  if (dc_conv_pairrows_supported(n, h, w, g)) return "k_conv_tc_pairrows";
  if (dc_conv_rows_supported(n, h, w, g)) return "k_conv_tc_rows";
  if (dc_conv_fold_supported(n, h, w, g)) return "k_conv_tc_fold";
  if (dc_conv_tc_supported(n, h, w, g)) return "k_conv_tc";
  if (dc_conv_stem_s2_supported(n, h, w, g) && dc_conv_stem_supported(n, h, w, g)) return "k_conv_stem_s2";
  if (dc_conv_stem_supported(n, h, w, g)) return "k_conv_stem_tc";
  if (dc_conv_smallcin_supported(n, h, w, g)) return "k_conv_smallcin_bf16";
  return "k_conv_dense_bf16";
}

extern "C" dc_status dc_conv_forward_algo(const void *x, int n, int h, int w, const dc_geom *g,
                                          const void *w_packed, const float *bias, dc_act act,
                                          const void *residual, void *y, dc_dtype dtype, void *workspace,
                                          size_t workspace_bytes, dc_stream stream, dc_algo algo) {
  dc_status s = dc_validate_geom(g);
  if (s != DC_OK) return s;
  if (g->groups != 1) return DC_ERR_UNSUPPORTED;  // depthwise layers go through dc_dwconv_forward
  if (!x || !y || !w_packed || n <= 0 || h <= 0 || w <= 0) return DC_ERR_INVALID_ARG;
  if (dtype != DC_F32 && dtype != DC_BF16) return DC_ERR_INVALID_ARG;
  if (act != DC_ACT_IDENTITY && act != DC_ACT_RELU6) return DC_ERR_INVALID_ARG;
  if (algo != DC_ALGO_AUTO && algo != DC_ALGO_TCGEN05 && algo != DC_ALGO_SIMT) return DC_ERR_INVALID_ARG;
  if (dc_out_extent(h, g->k, g->stride, g->pad) <= 0 || dc_out_extent(w, g->k, g->stride, g->pad) <= 0)
    return DC_ERR_SHAPE;
  if (!workspace || workspace_bytes < dc_conv_workspace_bytes()) return DC_ERR_WORKSPACE;
  if (!dc_aligned16(x) || !dc_aligned16(y) || !dc_aligned16(w_packed) || !dc_aligned16(workspace) ||
      (bias && !dc_aligned16(bias)) || (residual && !dc_aligned16(residual)))
    return DC_ERR_ALIGNMENT;
  cudaStream_t st = (cudaStream_t)stream;
  if (dtype == DC_BF16 && algo != DC_ALGO_SIMT && dc_conv_pairrows_supported(n, h, w, g))
    return dc_launch_conv_pairrows(x, n, h, w, g, w_packed, bias, act, residual, y, workspace, st);
  if (dtype == DC_BF16 && algo != DC_ALGO_SIMT && dc_conv_rows_supported(n, h, w, g))
    return dc_launch_conv_rows(x, n, h, w, g, w_packed, bias, act, residual, y, workspace, st);
  const bool fold_ok = dtype == DC_BF16 && dc_conv_fold_supported(n, h, w, g);
  const bool tc_ok = dtype == DC_BF16 && !fold_ok && dc_conv_tc_supported(n, h, w, g);
  const bool stem_ok = dtype == DC_BF16 && !fold_ok && !tc_ok && dc_conv_stem_supported(n, h, w, g);
  if (algo == DC_ALGO_TCGEN05 && !tc_ok && !fold_ok && !stem_ok) return DC_ERR_UNSUPPORTED;
  if (fold_ok && algo != DC_ALGO_SIMT)
    return dc_launch_conv_fold(x, n, h, w, g, w_packed, bias, act, residual, y, workspace, st);
  if (tc_ok && algo != DC_ALGO_SIMT)
    return dc_launch_conv_tc(x, n, h, w, g, w_packed, bias, act, residual, y, workspace, st);
  if (stem_ok && algo != DC_ALGO_SIMT && dc_conv_stem_s2_supported(n, h, w, g))
    return dc_launch_conv_stem_s2(x, n, h, w, g, w_packed, bias, act, residual, y, workspace, st);
  if (stem_ok && algo != DC_ALGO_SIMT)
    return dc_launch_conv_stem(x, n, h, w, g, w_packed, bias, act, residual, y, workspace, st);
  return dc_launch_conv_simt(x, n, h, w, g, w_packed, bias, act, residual, y, dtype, st);
}

extern "C" dc_status dc_conv_forward(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                                     const float *bias, dc_act act, const void *residual, void *y,
                                     dc_dtype dtype, void *workspace, size_t workspace_bytes, dc_stream stream) {
  return dc_conv_forward_algo(x, n, h, w, g, w_packed, bias, act, residual, y, dtype, workspace, workspace_bytes,
                              stream, DC_ALGO_AUTO);
}

extern "C" dc_status dc_workspace_status_where(void *workspace, dc_stream stream, unsigned int *where,
                                               unsigned int *detail) {
  if (!workspace) return DC_ERR_WORKSPACE;
  DC_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  unsigned int head[3] = {0, 0, 0};                    // status, site of the wait, first detail word
  DC_CUDA_OK(cudaMemcpy(head, workspace, sizeof(head), cudaMemcpyDeviceToHost));
  if (where) *where = head[1];
  if (detail) *detail = head[2];
  if (head[0] != 0) {
    DC_CUDA_OK(cudaMemset(workspace, 0, sizeof(DcWsHeader)));
    return DC_ERR_TIMEOUT;
  }
  return DC_OK;
}

extern "C" dc_status dc_workspace_status(void *workspace, dc_stream stream) {
  return dc_workspace_status_where(workspace, stream, nullptr, nullptr);
}

// ----------------------------------------------------------------------------------------------
// unmerged inverted-residual block: three launches sharing the caller's workspace
//   [status header][expand output n*h*w*c_hidden][depthwise output n*ho*wo*c_hidden]
// ----------------------------------------------------------------------------------------------
static dc_status check_block(int n, int h, int w, const dc_block *b, dc_dtype dtype) {
  if (!b || n <= 0 || h <= 0 || w <= 0) return DC_ERR_INVALID_ARG;
  if (dtype != DC_F32 && dtype != DC_BF16) return DC_ERR_INVALID_ARG;
  if (b->c_in <= 0 || b->c_hidden <= 0 || b->c_out <= 0 || b->dw_k <= 0 || b->dw_stride <= 0 || b->dw_pad < 0)
    return DC_ERR_INVALID_ARG;
  if (b->dw_k % 2 == 0) return DC_ERR_UNSUPPORTED;
  if (!b->has_expand && b->c_hidden != b->c_in) return DC_ERR_SHAPE;
  if (b->has_residual && (b->dw_stride != 1 || b->c_in != b->c_out || 2 * b->dw_pad != b->dw_k - 1))
    return DC_ERR_NOT_MERGEABLE;
  if (dc_out_extent(h, b->dw_k, b->dw_stride, b->dw_pad) <= 0 || dc_out_extent(w, b->dw_k, b->dw_stride, b->dw_pad) <= 0)
    return DC_ERR_SHAPE;
  return DC_OK;
}

extern "C" dc_status dc_block_workspace_bytes(int n, int h, int w, const dc_block *b, dc_dtype dtype,
                                              size_t *bytes) {
  dc_status s = check_block(n, h, w, b, dtype);
  if (s != DC_OK) return s;
  if (!bytes) return DC_ERR_INVALID_ARG;
  const size_t es = dtype == DC_F32 ? 4 : 2;
  const int ho = dc_out_extent(h, b->dw_k, b->dw_stride, b->dw_pad), wo = dc_out_extent(w, b->dw_k, b->dw_stride, b->dw_pad);
  size_t t = sizeof(DcWsHeader);
  if (b->has_expand) t += dc_round_up((size_t)n * h * w * b->c_hidden * es, 256);
  t += dc_round_up((size_t)n * ho * wo * b->c_hidden * es, 256);
  *bytes = t;
  return DC_OK;
}

extern "C" dc_status dc_block_forward(const void *x, int n, int h, int w, const dc_block *b, void *y,
                                      dc_dtype dtype, void *workspace, size_t workspace_bytes,
                                      dc_stream stream) {
  size_t need = 0;
  dc_status s = dc_block_workspace_bytes(n, h, w, b, dtype, &need);
  if (s != DC_OK) return s;
  if (!x || !y || !b->w_dw || !b->w_project || (b->has_expand && !b->w_expand)) return DC_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < need) return DC_ERR_WORKSPACE;
  if (!dc_aligned16(workspace)) return DC_ERR_ALIGNMENT;
  const size_t es = dtype == DC_F32 ? 4 : 2;
  const int ho = dc_out_extent(h, b->dw_k, b->dw_stride, b->dw_pad), wo = dc_out_extent(w, b->dw_k, b->dw_stride, b->dw_pad);
  char *ws = (char *)workspace;
  char *t_exp = ws + sizeof(DcWsHeader);
  char *t_dw = t_exp + (b->has_expand ? dc_round_up((size_t)n * h * w * b->c_hidden * es, 256) : 0);
  const void *dw_in = x;
  if (b->has_expand) {
    dc_geom ge = {b->c_in, b->c_hidden, 1, 1, 1, 0};
    s = dc_conv_forward(x, n, h, w, &ge, b->w_expand, b->b_expand, b->act_expand, nullptr, t_exp, dtype, ws,
                        sizeof(DcWsHeader), stream);
    if (s != DC_OK) return s;
    dw_in = t_exp;
  }
  s = dc_dwconv_forward(dw_in, n, h, w, b->c_hidden, b->dw_k, b->dw_stride, b->dw_pad, b->w_dw, b->b_dw, b->act_dw,
                        t_dw, dtype, stream);
  if (s != DC_OK) return s;
  dc_geom gp = {b->c_hidden, b->c_out, 1, 1, 1, 0};
  return dc_conv_forward(t_dw, n, ho, wo, &gp, b->w_project, b->b_project, DC_ACT_IDENTITY,
                         b->has_residual ? x : nullptr, y, dtype, ws, sizeof(DcWsHeader), stream);
}

// ----------------------------------------------------------------------------------------------
// whole path from host buffers
// ----------------------------------------------------------------------------------------------
struct HostPlan {
  dc_geom mg;
  size_t merge_ws, packed, x_bytes, y_bytes, params, total;
  int ho, wo;
};

static size_t layer_weight_elems(const dc_layer &L) {
  return (size_t)L.c_out * (L.c_in / L.groups) * L.k * L.k;
}

static dc_status host_plan(const dc_layer *layers, int nl, const dc_residual *res, int n_res, int n, int h, int w,
                           dc_dtype dtype, HostPlan *hp) {
  if (n <= 0 || h <= 0 || w <= 0) return DC_ERR_INVALID_ARG;
  if (dtype != DC_F32 && dtype != DC_BF16) return DC_ERR_INVALID_ARG;
  dc_status s = dc_merge_query(layers, nl, res, n_res, &hp->mg, &hp->merge_ws);
  if (s != DC_OK) return s;
  s = dc_packed_bytes(&hp->mg, dtype, &hp->packed);
  if (s != DC_OK) return s;
  hp->ho = dc_out_extent(h, hp->mg.k, hp->mg.stride, hp->mg.pad);
  hp->wo = dc_out_extent(w, hp->mg.k, hp->mg.stride, hp->mg.pad);
  if (hp->ho <= 0 || hp->wo <= 0) return DC_ERR_SHAPE;
  const size_t es = dtype == DC_F32 ? 4 : 2;
  hp->x_bytes = (size_t)n * h * w * hp->mg.c_in * es;
  hp->y_bytes = (size_t)n * hp->ho * hp->wo * hp->mg.c_out * es;
  size_t p = 0;
  for (int i = 0; i < nl; ++i) {
    p += dc_round_up(layer_weight_elems(layers[i]) * 4, 256);
    p += 5 * dc_round_up((size_t)layers[i].c_out * 4, 256);
  }
  hp->params = p;
  size_t mw = (size_t)hp->mg.c_out * hp->mg.c_in * hp->mg.k * hp->mg.k * 4;
  hp->total = sizeof(DcWsHeader) + p + dc_round_up(hp->merge_ws, 256) + dc_round_up(mw, 256) +
              dc_round_up((size_t)hp->mg.c_out * 4, 256) + dc_round_up(hp->packed, 256) +
              dc_round_up(hp->x_bytes, 256) + dc_round_up(hp->y_bytes, 256);
  return DC_OK;
}

extern "C" dc_status dc_chain_host_workspace_bytes(const dc_layer *layers, int n_layers, const dc_residual *res,
                                                   int n_res, int n, int h, int w, dc_dtype dtype, size_t *bytes) {
  HostPlan hp;
  dc_status s = host_plan(layers, n_layers, res, n_res, n, h, w, dtype, &hp);
  if (s != DC_OK) return s;
  if (!bytes) return DC_ERR_INVALID_ARG;
  *bytes = hp.total;
  return DC_OK;
}

extern "C" dc_status dc_chain_host_param_layout(const dc_layer *layers, int n_layers, size_t *offsets, size_t *total) {
  if (!layers || n_layers <= 0 || !total) return DC_ERR_INVALID_ARG;
  size_t o = 0;
  for (int i = 0; i < n_layers; ++i) {
    const dc_layer &L = layers[i];
    if (L.c_in <= 0 || L.c_out <= 0 || L.groups <= 0 || L.k <= 0 || L.c_in % L.groups) return DC_ERR_INVALID_ARG;
    for (int j = 0; j < 6; ++j) {
      if (offsets) offsets[6 * i + j] = o;
      o += dc_round_up(j == 0 ? layer_weight_elems(L) * 4 : (size_t)L.c_out * 4, 256);
    }
  }
  *total = o;
  return DC_OK;
}

extern "C" dc_status dc_chain_forward_host_async(const dc_layer *layers, int n_layers, const dc_residual *res,
                                                 int n_res, const void *x_host, int n, int h, int w, dc_act act,
                                                 void *y_host, dc_dtype dtype, void *workspace,
                                                 size_t workspace_bytes, dc_stream stream) {
  HostPlan hp;
  dc_status s = host_plan(layers, n_layers, res, n_res, n, h, w, dtype, &hp);
  if (s != DC_OK) return s;
  if (!x_host || !y_host) return DC_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < hp.total) return DC_ERR_WORKSPACE;
  if (!dc_aligned16(workspace)) return DC_ERR_ALIGNMENT;
  cudaStream_t st = (cudaStream_t)stream;
  char *base = (char *)workspace;
  size_t off = sizeof(DcWsHeader);
  auto take = [&](size_t bytes) { char *p = base + off; off += dc_round_up(bytes, 256); return p; };
  std::vector<dc_layer> dev(layers, layers + n_layers);
  // Device layout of the parameters: per layer the weights and the five vectors, each rounded up to
  // 256 bytes (dc_chain_host_param_layout).  When the caller's host arrays already lie in one block
  // in that layout, one copy moves them all; otherwise one copy per array.
  char *params_dev = base + off;
  const char *host_base = (const char *)layers[0].weight;
  bool one_block = host_base != nullptr;
  size_t last_end = 0;
  {
    size_t o = 0;
    for (int i = 0; i < n_layers && one_block; ++i) {
      const dc_layer &L = layers[i];
      const size_t wb = layer_weight_elems(L) * 4, cb = (size_t)L.c_out * 4;
      const float *src[6] = {L.weight, L.bias, L.bn_gamma, L.bn_beta, L.bn_mean, L.bn_var};
      for (int j = 0; j < 6; ++j) {
        const size_t bytes = j == 0 ? wb : cb;
        if (src[j]) {
          if ((const char *)src[j] != host_base + o) { one_block = false; break; }
          last_end = o + bytes;
        }
        o += dc_round_up(bytes, 256);
      }
    }
  }
  if (one_block) DC_CUDA_OK(cudaMemcpyAsync(params_dev, host_base, last_end, cudaMemcpyHostToDevice, st));
  for (int i = 0; i < n_layers; ++i) {
    const dc_layer &L = layers[i];
    size_t wb = layer_weight_elems(L) * 4, cb = (size_t)L.c_out * 4;
    float *dw = (float *)take(wb);
    if (!L.weight) return DC_ERR_INVALID_ARG;
    if (!one_block) DC_CUDA_OK(cudaMemcpyAsync(dw, L.weight, wb, cudaMemcpyHostToDevice, st));
    dev[i].weight = dw;
    const float *src[5] = {L.bias, L.bn_gamma, L.bn_beta, L.bn_mean, L.bn_var};
    const float **dst[5] = {&dev[i].bias, &dev[i].bn_gamma, &dev[i].bn_beta, &dev[i].bn_mean, &dev[i].bn_var};
    for (int j = 0; j < 5; ++j) {
      float *d = (float *)take(cb);
      if (src[j]) {
        if (!one_block) DC_CUDA_OK(cudaMemcpyAsync(d, src[j], cb, cudaMemcpyHostToDevice, st));
        *dst[j] = d;
      } else {
        *dst[j] = nullptr;
      }
    }
  }
  char *merge_ws = take(hp.merge_ws);
  float *w_merged = (float *)take((size_t)hp.mg.c_out * hp.mg.c_in * hp.mg.k * hp.mg.k * 4);
  float *b_merged = (float *)take((size_t)hp.mg.c_out * 4);
  char *packed = take(hp.packed);
  char *dx = take(hp.x_bytes);
  char *dy = take(hp.y_bytes);
  DC_CUDA_OK(cudaMemcpyAsync(dx, x_host, hp.x_bytes, cudaMemcpyHostToDevice, st));
  s = dc_merge_chain(dev.data(), n_layers, res, n_res, w_merged, b_merged, packed, dtype, merge_ws, hp.merge_ws,
                     stream);
  if (s != DC_OK) return s;
  s = dc_conv_forward(dx, n, h, w, &hp.mg, packed, b_merged, act, nullptr, dy, dtype, workspace, sizeof(DcWsHeader),
                      stream);
  if (s != DC_OK) return s;
  DC_CUDA_OK(cudaMemcpyAsync(y_host, dy, hp.y_bytes, cudaMemcpyDeviceToHost, st));
  return DC_OK;
}

extern "C" dc_status dc_chain_forward_host(const dc_layer *layers, int n_layers, const dc_residual *res, int n_res,
                                           const void *x_host, int n, int h, int w, dc_act act, void *y_host,
                                           dc_dtype dtype, void *workspace, size_t workspace_bytes,
                                           dc_stream stream) {
  dc_status s = dc_chain_forward_host_async(layers, n_layers, res, n_res, x_host, n, h, w, act, y_host, dtype,
                                            workspace, workspace_bytes, stream);
  if (s != DC_OK) return s;
  DC_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  return DC_OK;
}
