// CUDA-core convolution kernels: the fp32 accuracy path of the dense convolution, a generic
// bf16 dense convolution for shapes the tensor-core kernel does not take, and the depthwise
// stencil.  NHWC, fp32 accumulation.
#include "common.cuh"

// ----------------------------------------------------------------------------------------------
// dense, fp32: one thread = one output pixel x 4 consecutive output channels.
// weights fp32 [k][k][c_in][c_out]: threads of a pixel read consecutive output channels.
// ----------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) k_conv_dense_f32(const float *__restrict__ x, const float *__restrict__ w,
                                                        const float *__restrict__ bias,
                                                        const float *__restrict__ residual, float *__restrict__ y,
                                                        int n, int h, int wd, int ho, int wo, dc_geom g, int act) {
  const int noc = (g.c_out + 3) / 4;
  const long long total = (long long)n * ho * wo * noc;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int oc = (int)(idx % noc) * 4;
    long long pix = idx / noc;
    const int X = (int)(pix % wo), Y = (int)((pix / wo) % ho), img = (int)(pix / ((long long)wo * ho));
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int u = 0; u < g.k; ++u) {
      const int yy = Y * g.stride + u - g.pad;
      if (yy < 0 || yy >= h) continue;
      for (int v = 0; v < g.k; ++v) {
        const int xx = X * g.stride + v - g.pad;
        if (xx < 0 || xx >= wd) continue;
        const float *xp = x + (((size_t)img * h + yy) * wd + xx) * g.c_in;
        const float *wp = w + ((size_t)(u * g.k + v) * g.c_in) * g.c_out + oc;
        for (int c = 0; c < g.c_in; ++c) {
          const float xv = xp[c];
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (oc + q < g.c_out) acc[q] = fmaf(xv, wp[(size_t)c * g.c_out + q], acc[q]);
        }
      }
    }
    const size_t obase = (((size_t)img * ho + Y) * wo + X) * g.c_out + oc;
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (oc + q < g.c_out) {
        float v = acc[q] + (bias ? bias[oc + q] : 0.f);
        if (residual) v += residual[obase + q];
        y[obase + q] = dc_act_apply(v, act);
      }
  }
}

// ----------------------------------------------------------------------------------------------
// dense, bf16 storage: one thread = one output pixel x one output channel; the packed weights
// are the chunk planes [plane][n_pad][8] of KOrder, so threads of a pixel read consecutive
// 16-byte chunks.  fp32 accumulation, one rounding at the store.
// ----------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) k_conv_dense_bf16(const __nv_bfloat16 *__restrict__ x,
                                                         const __nv_bfloat16 *__restrict__ w,
                                                         const float *__restrict__ bias,
                                                         const __nv_bfloat16 *__restrict__ residual,
                                                         __nv_bfloat16 *__restrict__ y, int n, int h, int wd,
                                                         int ho, int wo, dc_geom g, KOrder ko, int act) {
  const long long total = (long long)n * ho * wo * g.c_out;
  const bool vec = (g.c_in % 8) == 0;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int o = (int)(idx % g.c_out);
    long long pix = idx / g.c_out;
    const int X = (int)(pix % wo), Y = (int)((pix / wo) % ho), img = (int)(pix / ((long long)wo * ho));
    float acc = 0.f;
    for (int u = 0; u < g.k; ++u) {
      const int yy = Y * g.stride + u - g.pad;
      if (yy < 0 || yy >= h) continue;
      for (int v = 0; v < g.k; ++v) {
        const int xx = X * g.stride + v - g.pad;
        if (xx < 0 || xx >= wd) continue;
        const __nv_bfloat16 *xp = x + (((size_t)img * h + yy) * wd + xx) * g.c_in;
        for (int cc = 0; cc < ko.cch; ++cc) {
          const int plane = dc_korder_encode(ko, cc, u, v);
          const uint4 wv = *reinterpret_cast<const uint4 *>(w + dc_packed_chunk(ko, plane, dc_korder_row(ko, v, o)) * 8);
          const __nv_bfloat16 *wb = reinterpret_cast<const __nv_bfloat16 *>(&wv);
          if (vec) {
            const uint4 xv = *reinterpret_cast<const uint4 *>(xp + cc * 8);
            const __nv_bfloat16 *xb = reinterpret_cast<const __nv_bfloat16 *>(&xv);
#pragma unroll
            for (int q = 0; q < 8; ++q) acc = fmaf(__bfloat162float(xb[q]), __bfloat162float(wb[q]), acc);
          } else {
#pragma unroll
            for (int q = 0; q < 8; ++q)
              if (cc * 8 + q < g.c_in) acc = fmaf(__bfloat162float(xp[cc * 8 + q]), __bfloat162float(wb[q]), acc);
          }
        }
      }
    }
    const size_t oi = (((size_t)img * ho + Y) * wo + X) * g.c_out + o;
    float vout = acc + (bias ? bias[o] : 0.f);
    if (residual) vout += __bfloat162float(residual[oi]);
    y[oi] = __float2bfloat16_rn(dc_act_apply(vout, act));
  }
}

static inline int simt_blocks(long long total, int threads, int cap) {
  long long b = (total + threads - 1) / threads;
  if (b > cap) b = cap;
  if (b < 1) b = 1;
  return (int)b;
}

// ----------------------------------------------------------------------------------------------
// dense conv with very few input channels (the 3-channel stem), bf16, fp32 accumulate.
// The reduction is only k*k*c_in long (27 for the stem), far too short and too ragged (6-byte
// pixels) for the tensor-core staging, and the layer is bound by writing its output.  Persistent
// CTAs walk output row segments of 128 pixels; one thread = one pixel x CO_T output channels:
//   * the k input rows of the segment are staged in shared memory with coalesced loads (zeros
//     outside the image), each thread then reads its k*k*c_in inputs from there;
//   * weights sit in shared memory as fp32 [tap][c][o]; every thread of a warp reads the same
//     address (a broadcast), four output channels per load;
//   * a thread's CO_T channels are 2*CO_T contiguous bytes of the NHWC output: 16-byte stores.
// ----------------------------------------------------------------------------------------------
constexpr int kSmallCinMax = 4;
constexpr int kSmallTile = 128;
constexpr int kSmallRows = 2;                    // output rows per thread

template <int CO_T>
__global__ void __launch_bounds__(kSmallTile)
k_conv_smallcin_bf16(const __nv_bfloat16 *__restrict__ x, const __nv_bfloat16 *__restrict__ w,
                     const float *__restrict__ bias, const __nv_bfloat16 *__restrict__ residual,
                     __nv_bfloat16 *__restrict__ y, int n, int h, int wd, int ho, int wo, dc_geom g, KOrder ko,
                     int act, int xtiles, int o0) {
  extern __shared__ __align__(16) unsigned char sm_raw[];
  const int taps = g.k * g.k;
  float *w_s = reinterpret_cast<float *>(sm_raw);                       // [taps][c_in][CO_T]
  float *b_s = w_s + taps * g.c_in * CO_T;                              // [CO_T]
  __nv_bfloat16 *x_s = reinterpret_cast<__nv_bfloat16 *>(b_s + CO_T);   // [(rows-1)*stride + k][span][c_in]
  const int span = (kSmallTile - 1) * g.stride + g.k;                   // input pixels per staged row
  const int row_elems = span * g.c_in;
  const int tid = (int)threadIdx.x;
  // weights and bias of this pass's CO_T output channels: once per CTA (CTAs are persistent)
  for (int i = tid; i < taps * g.c_in * CO_T; i += kSmallTile) {
    const int o = i % CO_T, c = (i / CO_T) % g.c_in, t = i / (CO_T * g.c_in);
    const int u = t / g.k, v = t - u * g.k;
    float wv = 0.f;
    if (o0 + o < g.c_out) {
      const int plane = dc_korder_encode(ko, c / 8, u, v);
      wv = __bfloat162float(w[dc_packed_chunk(ko, plane, dc_korder_row(ko, v, o0 + o)) * 8 + (c & 7)]);
    }
    w_s[i] = wv;
  }
  if (tid < CO_T) b_s[tid] = (bias && o0 + tid < g.c_out) ? bias[o0 + tid] : 0.f;
  // a tile = kSmallRows output rows x 128 pixels; a thread computes its pixel in each of the rows,
  // so every weight vector it reads from shared memory feeds kSmallRows x 4 FMAs
  const int ypairs = (ho + kSmallRows - 1) / kSmallRows;
  const int srows = (kSmallRows - 1) * g.stride + g.k;                  // staged input rows
  const long long total = (long long)n * ypairs * xtiles;
  for (long long tile = blockIdx.x; tile < total; tile += gridDim.x) {
    const int xt = (int)(tile % xtiles);
    const long long rowi = tile / xtiles;
    const int Y0 = (int)(rowi % ypairs) * kSmallRows, img = (int)(rowi / ypairs);
    const int X0 = xt * kSmallTile;
    const int gx0 = X0 * g.stride - g.pad, gy0 = Y0 * g.stride - g.pad;
    __syncthreads();                              // weights staged / previous tile done with x_s
    // stage the input rows of the tile: thread = pixel, contiguous along the row
    for (int r = 0; r < srows; ++r) {
      const int gy = gy0 + r;
      const bool rok = gy >= 0 && gy < h;
      const __nv_bfloat16 *src = x + (((size_t)img * h + (rok ? gy : 0)) * wd) * g.c_in;
      for (int px = tid; px < span; px += kSmallTile) {
        const int gx = gx0 + px;
        const bool ok = rok && gx >= 0 && gx < wd;
        for (int c = 0; c < g.c_in; ++c)
          x_s[r * row_elems + px * g.c_in + c] = ok ? src[(size_t)gx * g.c_in + c] : __float2bfloat16_rn(0.f);
      }
    }
    __syncthreads();
    const int X = X0 + tid;
    if (X < wo) {
      float acc[kSmallRows][CO_T];
#pragma unroll
      for (int j = 0; j < kSmallRows; ++j)
#pragma unroll
        for (int o = 0; o < CO_T; ++o) acc[j][o] = b_s[o];
      const __nv_bfloat16 *xp = x_s + tid * g.stride * g.c_in;
      const float *wp = w_s;
      for (int u = 0; u < g.k; ++u, xp += row_elems - g.k * g.c_in) {
        for (int vc = 0; vc < g.k * g.c_in; ++vc, ++xp, wp += CO_T) {
          float xv[kSmallRows];
#pragma unroll
          for (int j = 0; j < kSmallRows; ++j) xv[j] = __bfloat162float(xp[j * g.stride * row_elems]);
#pragma unroll
          for (int o = 0; o < CO_T; o += 4) {
            const float4 w4 = *reinterpret_cast<const float4 *>(wp + o);
#pragma unroll
            for (int j = 0; j < kSmallRows; ++j) {
              acc[j][o] = fmaf(xv[j], w4.x, acc[j][o]); acc[j][o + 1] = fmaf(xv[j], w4.y, acc[j][o + 1]);
              acc[j][o + 2] = fmaf(xv[j], w4.z, acc[j][o + 2]); acc[j][o + 3] = fmaf(xv[j], w4.w, acc[j][o + 3]);
            }
          }
        }
      }
#pragma unroll
      for (int j = 0; j < kSmallRows; ++j) {
        const size_t oi = (((size_t)img * ho + (Y0 + j)) * wo + X) * g.c_out + o0;
#pragma unroll
        for (int o = 0; o < CO_T; o += 8) {
          if (Y0 + j < ho && o0 + o < g.c_out) {  // c_out is a multiple of 8
            if (residual) {
              const uint4 rv = *reinterpret_cast<const uint4 *>(residual + oi + o);
              const __nv_bfloat162 *rb = reinterpret_cast<const __nv_bfloat162 *>(&rv);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float2 rf = __bfloat1622float2(rb[i]);
                acc[j][o + 2 * i] += rf.x; acc[j][o + 2 * i + 1] += rf.y;
              }
            }
            uint4 ov;
            __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              ob[i] = __floats2bfloat162_rn(dc_act_apply(acc[j][o + 2 * i], act), dc_act_apply(acc[j][o + 2 * i + 1], act));
            *reinterpret_cast<uint4 *>(y + oi + o) = ov;
          }
        }
      }
    }
  }
}

static bool smallcin_ok(const dc_geom *g) {
  return g->groups == 1 && g->c_in <= kSmallCinMax && g->c_out % 8 == 0 && g->k <= 5 && g->stride <= 2;
}

bool dc_conv_smallcin_supported(int n, int h, int w, const dc_geom *g) {
  (void)n; (void)h; (void)w;
  return smallcin_ok(g);
}

dc_status dc_launch_conv_simt(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                              const float *bias, dc_act act, const void *residual, void *y,
                              dc_dtype dtype, cudaStream_t stream) {
  const int ho = dc_out_extent(h, g->k, g->stride, g->pad), wo = dc_out_extent(w, g->k, g->stride, g->pad);
  if (dtype == DC_F32) {
    long long total = (long long)n * ho * wo * ((g->c_out + 3) / 4);
    k_conv_dense_f32<<<simt_blocks(total, 128, 148 * 64), 128, 0, stream>>>(
        (const float *)x, (const float *)w_packed, bias, (const float *)residual, (float *)y, n, h, w, ho, wo, *g,
        (int)act);
  } else {
    KOrder ko;
    dc_korder_init(&ko, g);
    if (smallcin_ok(g)) {
      constexpr int CO_T = 32;
      const int xtiles = dc_div_up(wo, kSmallTile);
      const int span = (kSmallTile - 1) * g->stride + g->k;
      const size_t smem = (size_t)(g->k * g->k * g->c_in * CO_T + CO_T) * 4 +
                          (size_t)((kSmallRows - 1) * g->stride + g->k) * span * g->c_in * 2;
      const long long tiles = (long long)n * dc_div_up(ho, kSmallRows) * xtiles;
      const int grid = (int)(tiles < 148 * 8 ? tiles : 148 * 8);      // persistent CTAs, 8 per SM
      for (int o0 = 0; o0 < g->c_out; o0 += CO_T)                      // one pass per 32 output channels
        k_conv_smallcin_bf16<CO_T><<<grid, kSmallTile, smem, stream>>>(
            (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w_packed, bias, (const __nv_bfloat16 *)residual,
            (__nv_bfloat16 *)y, n, h, w, ho, wo, *g, ko, (int)act, xtiles, o0);
      return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
    }
    long long total = (long long)n * ho * wo * g->c_out;
    k_conv_dense_bf16<<<simt_blocks(total, 128, 148 * 64), 128, 0, stream>>>(
        (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w_packed, bias, (const __nv_bfloat16 *)residual,
        (__nv_bfloat16 *)y, n, h, w, ho, wo, *g, ko, (int)act);
  }
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}

// ----------------------------------------------------------------------------------------------
// depthwise stencil.  One thread = one output pixel x VEC consecutive channels (16 bytes of
// storage: 8 bf16 or 4 fp32), so a warp reads and writes whole 128-byte lines of the NHWC map.
// weights fp32 [k][k][c].
// ----------------------------------------------------------------------------------------------
template <typename T> struct DwVec;
template <> struct DwVec<float> {
  static constexpr int V = 4;
  __device__ static void load(const float *p, float *o) {
    float4 v = *reinterpret_cast<const float4 *>(p);
    o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
  }
  __device__ static void store(float *p, const float *o) {
    *reinterpret_cast<float4 *>(p) = make_float4(o[0], o[1], o[2], o[3]);
  }
  __device__ static float ld1(const float *p) { return *p; }
  __device__ static void st1(float *p, float v) { *p = v; }
};
template <> struct DwVec<__nv_bfloat16> {
  static constexpr int V = 8;
  __device__ static void load(const __nv_bfloat16 *p, float *o) {
    uint4 v = *reinterpret_cast<const uint4 *>(p);
    const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
    for (int q = 0; q < 4; ++q) { float2 f = __bfloat1622float2(b[q]); o[2 * q] = f.x; o[2 * q + 1] = f.y; }
  }
  __device__ static void store(__nv_bfloat16 *p, const float *o) {
    uint4 v;
    __nv_bfloat162 *b = reinterpret_cast<__nv_bfloat162 *>(&v);
#pragma unroll
    for (int q = 0; q < 4; ++q) b[q] = __floats2bfloat162_rn(o[2 * q], o[2 * q + 1]);
    *reinterpret_cast<uint4 *>(p) = v;
  }
  __device__ static float ld1(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
  __device__ static void st1(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }
};

template <typename T>
__global__ void __launch_bounds__(256) k_dwconv_vec(const T *__restrict__ x, const float *__restrict__ w,
                                                    const float *__restrict__ bias, T *__restrict__ y, int n, int h,
                                                    int wd, int c, int ho, int wo, int k, int stride, int pad,
                                                    int act) {
  constexpr int V = DwVec<T>::V;
  const int cv = c / V;
  const long long total = (long long)n * ho * wo * cv;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int c0 = (int)(idx % cv) * V;
    long long pix = idx / cv;
    const int X = (int)(pix % wo), Y = (int)((pix / wo) % ho), img = (int)(pix / ((long long)wo * ho));
    float acc[V];
#pragma unroll
    for (int q = 0; q < V; ++q) acc[q] = bias ? bias[c0 + q] : 0.f;
    for (int u = 0; u < k; ++u) {
      const int yy = Y * stride + u - pad;
      if (yy < 0 || yy >= h) continue;
      for (int v = 0; v < k; ++v) {
        const int xx = X * stride + v - pad;
        if (xx < 0 || xx >= wd) continue;
        float xv[V];
        DwVec<T>::load(x + (((size_t)img * h + yy) * wd + xx) * c + c0, xv);
        const float *wp = w + (size_t)(u * k + v) * c + c0;
#pragma unroll
        for (int q = 0; q < V; q += 4) {
          const float4 wv = *reinterpret_cast<const float4 *>(wp + q);
          acc[q] = fmaf(xv[q], wv.x, acc[q]);
          acc[q + 1] = fmaf(xv[q + 1], wv.y, acc[q + 1]);
          acc[q + 2] = fmaf(xv[q + 2], wv.z, acc[q + 2]);
          acc[q + 3] = fmaf(xv[q + 3], wv.w, acc[q + 3]);
        }
      }
    }
#pragma unroll
    for (int q = 0; q < V; ++q) acc[q] = dc_act_apply(acc[q], act);
    DwVec<T>::store(y + (((size_t)img * ho + Y) * wo + X) * c + c0, acc);
  }
}

// Register-tiled variant for the common shapes (k = 3 or 5, stride 1 or 2): a CTA works on one
// output row, a thread on TX consecutive outputs x V channels, so the (TX-1)*S + K input vectors of
// a tap row are loaded once and reused by all the outputs they reach, and the tap row's weights are
// loaded once per TX outputs.  All index arithmetic is 32-bit and per row.
template <typename T, int K, int S, int TX>
__global__ void __launch_bounds__(128) k_dwconv_rows(const T *__restrict__ x, const float *__restrict__ w,
                                                     const float *__restrict__ bias, T *__restrict__ y, int h, int wd,
                                                     int c, int ho, int wo, int pad, int act) {
  constexpr int V = DwVec<T>::V;
  constexpr int NJ = (TX - 1) * S + K;
  const int cv = c / V;
  const int xtiles = (wo + TX - 1) / TX;
  const int row = (int)blockIdx.x;               // img * ho + Y
  const int img = row / ho, Y = row - img * ho;
  const T *ximg = x + (size_t)img * h * wd * c;
  T *yrow = y + (size_t)row * wo * c;
  for (int item = (int)threadIdx.x; item < xtiles * cv; item += (int)blockDim.x) {
    const int xt = item / cv, c0 = (item - xt * cv) * V;
    const int X0 = xt * TX;
    float acc[TX][V];
#pragma unroll
    for (int q = 0; q < V; ++q) {
      const float b = bias ? bias[c0 + q] : 0.f;
#pragma unroll
      for (int t = 0; t < TX; ++t) acc[t][q] = b;
    }
#pragma unroll
    for (int r = 0; r < K; ++r) {
      const int yy = Y * S + r - pad;
      if (yy < 0 || yy >= h) continue;
      float wr[K][V];
#pragma unroll
      for (int sx = 0; sx < K; ++sx) {
        const float *wp = w + (size_t)(r * K + sx) * c + c0;
#pragma unroll
        for (int q = 0; q < V; q += 4) {
          const float4 wv = *reinterpret_cast<const float4 *>(wp + q);
          wr[sx][q] = wv.x; wr[sx][q + 1] = wv.y; wr[sx][q + 2] = wv.z; wr[sx][q + 3] = wv.w;
        }
      }
      const T *xrow = ximg + (size_t)yy * wd * c + c0;
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const int xx = X0 * S + j - pad;
        float xv[V];
        if (xx >= 0 && xx < wd) {
          DwVec<T>::load(xrow + (size_t)xx * c, xv);
        } else {
#pragma unroll
          for (int q = 0; q < V; ++q) xv[q] = 0.f;
        }
#pragma unroll
        for (int t = 0; t < TX; ++t) {
          const int sx = j - t * S;                // tap column with which input j feeds output t
          if (sx >= 0 && sx < K) {
#pragma unroll
            for (int q = 0; q < V; ++q) acc[t][q] = fmaf(xv[q], wr[sx][q], acc[t][q]);
          }
        }
      }
    }
#pragma unroll
    for (int t = 0; t < TX; ++t) {
      if (X0 + t < wo) {
#pragma unroll
        for (int q = 0; q < V; ++q) acc[t][q] = dc_act_apply(acc[t][q], act);
        DwVec<T>::store(yrow + (size_t)(X0 + t) * c + c0, acc[t]);
      }
    }
  }
}

// any channel count: one thread = one output element
template <typename T>
__global__ void k_dwconv_scalar(const T *__restrict__ x, const float *__restrict__ w, const float *__restrict__ bias,
                                T *__restrict__ y, int n, int h, int wd, int c, int ho, int wo, int k, int stride,
                                int pad, int act) {
  const long long total = (long long)n * ho * wo * c;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int ch = (int)(idx % c);
    long long pix = idx / c;
    const int X = (int)(pix % wo), Y = (int)((pix / wo) % ho), img = (int)(pix / ((long long)wo * ho));
    float acc = bias ? bias[ch] : 0.f;
    for (int u = 0; u < k; ++u) {
      const int yy = Y * stride + u - pad;
      if (yy < 0 || yy >= h) continue;
      for (int v = 0; v < k; ++v) {
        const int xx = X * stride + v - pad;
        if (xx < 0 || xx >= wd) continue;
        acc = fmaf(DwVec<T>::ld1(x + (((size_t)img * h + yy) * wd + xx) * c + ch), w[(size_t)(u * k + v) * c + ch], acc);
      }
    }
    DwVec<T>::st1(y + idx, dc_act_apply(acc, act));
  }
}

template <typename T>
static dc_status launch_dw(const void *x, int n, int h, int w, int c, int k, int stride, int pad, const float *wp,
                           const float *bias, dc_act act, void *y, cudaStream_t st) {
  const int ho = dc_out_extent(h, k, stride, pad), wo = dc_out_extent(w, k, stride, pad);
  constexpr int V = DwVec<T>::V;
  // bf16, common shapes: the shared-memory stencil (TMA-staged haloed tile)
  if (sizeof(T) == 2 && dc_dwconv_stencil_supported(n, h, w, c, k, stride, pad))
    return dc_launch_dwconv_stencil(x, n, h, w, c, k, stride, pad, wp, bias, act, y, st);
  if (c % V == 0 && (k == 3 || k == 5) && (stride == 1 || stride == 2) && (long long)n * ho < (1ll << 31)) {
    // stride 1: 4 outputs per thread share 6 (k = 3) input columns; stride 2 shares less, so 2 outputs
    // keep the register count down.  Threads per CTA: the row's work items, in whole warps, up to 128.
    const int rows = n * ho;
    const T *xp = (const T *)x;
    T *yp = (T *)y;
    const int tx = stride == 1 ? 4 : 2;
    int items = dc_div_up(wo, tx) * (c / V);
    int threads = items >= 128 ? 128 : (int)dc_round_up((size_t)items, 32);
    if (k == 3 && stride == 1) k_dwconv_rows<T, 3, 1, 4><<<rows, threads, 0, st>>>(xp, wp, bias, yp, h, w, c, ho, wo, pad, (int)act);
    else if (k == 3) k_dwconv_rows<T, 3, 2, 2><<<rows, threads, 0, st>>>(xp, wp, bias, yp, h, w, c, ho, wo, pad, (int)act);
    else if (stride == 1) k_dwconv_rows<T, 5, 1, 4><<<rows, threads, 0, st>>>(xp, wp, bias, yp, h, w, c, ho, wo, pad, (int)act);
    else k_dwconv_rows<T, 5, 2, 2><<<rows, threads, 0, st>>>(xp, wp, bias, yp, h, w, c, ho, wo, pad, (int)act);
  } else if (c % V == 0) {
    long long total = (long long)n * ho * wo * (c / V);
    k_dwconv_vec<T><<<simt_blocks(total, 256, 148 * 32), 256, 0, st>>>((const T *)x, wp, bias, (T *)y, n, h, w, c, ho,
                                                                      wo, k, stride, pad, (int)act);
  } else {
    long long total = (long long)n * ho * wo * c;
    k_dwconv_scalar<T><<<simt_blocks(total, 256, 148 * 32), 256, 0, st>>>((const T *)x, wp, bias, (T *)y, n, h, w, c,
                                                                         ho, wo, k, stride, pad, (int)act);
  }
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}

extern "C" dc_status dc_dwconv_forward(const void *x, int n, int h, int w, int c, int k, int stride, int pad,
                                       const float *w_packed, const float *bias, dc_act act, void *y,
                                       dc_dtype dtype, dc_stream stream) {
  if (!x || !y || !w_packed) return DC_ERR_INVALID_ARG;
  if (n <= 0 || h <= 0 || w <= 0 || c <= 0 || k <= 0 || stride <= 0 || pad < 0) return DC_ERR_INVALID_ARG;
  if (dtype != DC_F32 && dtype != DC_BF16) return DC_ERR_INVALID_ARG;
  if (act != DC_ACT_IDENTITY && act != DC_ACT_RELU6) return DC_ERR_INVALID_ARG;
  if (k % 2 == 0) return DC_ERR_UNSUPPORTED;
  if (dc_out_extent(h, k, stride, pad) <= 0 || dc_out_extent(w, k, stride, pad) <= 0) return DC_ERR_SHAPE;
  if (!dc_aligned16(x) || !dc_aligned16(y) || !dc_aligned16(w_packed) || (bias && !dc_aligned16(bias)))
    return DC_ERR_ALIGNMENT;
  if (dtype == DC_F32)
    return launch_dw<float>(x, n, h, w, c, k, stride, pad, w_packed, bias, act, y, (cudaStream_t)stream);
  return launch_dw<__nv_bfloat16>(x, n, h, w, c, k, stride, pad, w_packed, bias, act, y, (cudaStream_t)stream);
}
