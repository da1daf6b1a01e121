// Depthwise convolution (bf16, k = 3 or 5, stride 1 or 2) as a shared-memory stencil on CUDA cores.
//
// A CTA owns a tile of output rows x the whole output width x a group of channels (x several
// images for small maps).  One 4-D TMA load brings the haloed input patch of the tile into shared
// memory as [image][row][column][channel]; the TMA unit writes zeros for everything outside the image,
// so the stencil itself has no border cases.  Threads then compute from shared memory: a thread owns
// 8 channels (one 16-byte vector) of TX neighbouring outputs of one row, so the (TX-1)*S + K input
// vectors of a tap row are read once for all the outputs they feed, with fp32 weights and fp32
// accumulation, and writes its results as 16-byte vectors (neighbouring threads write neighbouring
// vectors of a pixel: whole 32-byte sectors).  Depthwise layers are bound by HBM (1.8-4.5 FLOP/B):
// the tile is read from HBM once (neighbouring tiles share only their halo rows), and several CTAs
// per SM overlap one tile's load with another's arithmetic and stores.  No tensor cores.
//
// The one wait (for the tile to land) is bounded like every wait of the library; a wait that runs
// out sets a library-wide flag that dc_dwconv_status reports, and the CTA returns.
#include "tc_ptx.cuh"

namespace {
using namespace tc;

constexpr int kThreads = 128;
constexpr int kV = 8;                            // channels per thread (16 bytes of bf16)
constexpr int kTileBytes = 48 * 1024;            // patch size limit: four CTAs per SM, so that three loads are in flight
                                                 // while one tile is computed (measured: 256 threads x 2 CTAs x 64 KB
                                                 // took 76 / 100 us on the 112 x 112 layers of cfg4, this 68 / 81 us)

struct StencilParams {
  int n_img, h, w, c, ho, wo, pad, act;
  int ct, cgroups;             // channels per tile, tiles per pixel's channels
  int rt, ytiles;              // output rows per tile, tiles per image column
  int ni, igroups;             // images per tile, tiles over the batch
  int in_rows, in_w;           // patch rows and columns (with halo)
  int box_bytes, patch_bytes;  // bytes the TMA load delivers; the same rounded up to 128
};

// Outputs of one row that a thread computes together (the kernel's register tile and the patch width depend on
// it).  Stride 1: an ODD count.  The two items of a quarter warp (4 lanes = the 64 bytes of a 32-channel pixel
// each) then read pixels of different parity, i.e. the two halves of the 128 bytes that the 32 banks span; with
// 8 outputs per item all eight items of a warp read from the same 16 banks and every 16-byte load took two
// wavefronts (112 x 112 x 32: 49 us with 8, 42 us with 7; 5x5 at 28 x 28 x 240: 96 us with 4, 48 us with 5).
// Stride 2 moves an item by an even number of pixels whatever the count.
__host__ __device__ constexpr int outputs_per_item(int k, int stride) {
  return stride == 1 ? (k == 3 ? 7 : 5) : (k == 3 ? 4 : 2);
}

__device__ unsigned int g_dw_status;             // DC_ERR_TIMEOUT once a wait of these kernels ran out

__device__ __forceinline__ float4 lds_f4(uint32_t a) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
  return v;
}

template <int K, int S, int ACT, int CT>
__global__ void __launch_bounds__(kThreads, 4)
k_dwconv_stencil(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ StencilParams p,
                 const float *__restrict__ w, const float *__restrict__ bias, __nv_bfloat16 *__restrict__ y) {
  constexpr int TX = outputs_per_item(K, S);
  constexpr int NJ = (TX - 1) * S + K;           // input columns they read
  // channels per tile: compile-time for the common 32 (every shared-memory offset of the stencil is then an
  // immediate of its load), run-time otherwise
  const int ct = CT ? CT : p.ct;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t abort_word;
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  float *w_s = reinterpret_cast<float *>(smem + p.patch_bytes);          // [K*K][ct] weights, then [ct] bias

  // tile of this CTA: (image group, row tile, channel group), channel groups fastest
  int t = (int)blockIdx.x;
  const int cg = t % p.cgroups; t /= p.cgroups;
  const int ty = t % p.ytiles;
  const int ig = t / p.ytiles;
  const int c0 = cg * ct, y0 = ty * p.rt, img0 = ig * p.ni;

  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_word = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  dc_pdl_enter();                                // nothing above touched global memory; everything below may
  if (threadIdx.x == 0) {
    mbar_arrive_expect_tx(&bar, (uint32_t)p.box_bytes);
    // coordinates may be negative or reach past the tensor: those elements arrive as zeros
    tma_load_4d(smem_u32(smem), &map_x, &bar, c0, -p.pad, y0 * S - p.pad, img0);
  }
  for (int i = (int)threadIdx.x; i < (K * K + 1) * ct; i += kThreads) {
    const int tap = i / ct, ch = i - tap * ct;
    w_s[i] = tap < K * K ? w[(size_t)tap * p.c + c0 + ch] : (bias ? bias[c0 + ch] : 0.f);
  }
  __syncthreads();
  if (!mbar_wait(&bar, 0, &abort_word, nullptr, 0xA0000u)) {
    atomicExch(&g_dw_status, (unsigned int)DC_ERR_TIMEOUT);
    return;
  }

  const int cvt = ct / kV;                       // vectors per pixel of this tile: divides kThreads
  const int cv = (int)threadIdx.x % cvt;         // this thread's vector, the same for all its items
  const int xtiles = (p.wo + TX - 1) / TX;
  const int rows_valid = p.ho - y0 < p.rt ? p.ho - y0 : p.rt;
  const int imgs_valid = p.n_img - img0 < p.ni ? p.n_img - img0 : p.ni;
  // shared-memory addresses as 32-bit offsets (the loop below is bound by its instruction stream)
  const uint32_t ct2 = (uint32_t)ct * 2u, ct4 = (uint32_t)ct * 4u;
  const uint32_t w_sa = smem_u32(w_s) + (uint32_t)(cv * kV) * 4u;         // this thread's 8 channels of tap 0
  const uint32_t row_pitch = (uint32_t)p.in_w * ct2, img_pitch = (uint32_t)p.in_rows * row_pitch;   // bytes
  const uint32_t patch_sa = smem_u32(smem) + (uint32_t)(cv * kV) * 2u;
  const size_t c2 = (size_t)p.c * 2;             // bytes from one output pixel to the next
  // items (image, row, group of TX outputs) of this thread: the first one by division, the following ones by
  // adding the decomposed step with carries (two divisions per item cost more than the rest of its index work)
  const int step = kThreads / cvt;
  const int d_il = step / (rows_valid * xtiles), d_rem = step - d_il * rows_valid * xtiles;
  const int d_ry = d_rem / xtiles, d_xt = d_rem - d_ry * xtiles;
  int il, ry, xt;
  {
    const int item = (int)threadIdx.x / cvt;
    il = item / (rows_valid * xtiles);
    const int rem = item - il * rows_valid * xtiles;
    ry = rem / xtiles;
    xt = rem - ry * xtiles;
  }
#pragma unroll 1
  while (il < imgs_valid) {
    const int X0 = xt * TX;
    // packed fp32 arithmetic (two multiply-adds per instruction): the layer has 4.5 FLOP per byte
    // moved, which one scalar FMA per instruction would not keep up with
    float2 acc[TX][kV / 2];
    float2 bz[kV / 2];
    {
      const float4 b0 = lds_f4(w_sa + (uint32_t)(K * K) * ct4), b1 = lds_f4(w_sa + (uint32_t)(K * K) * ct4 + 16u);
      bz[0] = make_float2(b0.x, b0.y); bz[1] = make_float2(b0.z, b0.w);
      bz[2] = make_float2(b1.x, b1.y); bz[3] = make_float2(b1.z, b1.w);
    }
    uint32_t prow = patch_sa + (uint32_t)il * img_pitch + (uint32_t)(ry * S) * row_pitch + (uint32_t)(X0 * S) * ct2;
    // tap rows unrolled: the first one starts every accumulator from the bias (no copy of it), and with a
    // compile-time tile width the weights' and inputs' offsets are immediates
#pragma unroll
    for (int r = 0; r < K; ++r, prow += row_pitch) {
      float2 wr[K][kV / 2];
#pragma unroll
      for (int sx = 0; sx < K; ++sx) {
        const uint32_t wa = w_sa + (uint32_t)(r * K + sx) * ct4;
        const float4 w0 = lds_f4(wa), w1 = lds_f4(wa + 16u);
        wr[sx][0] = make_float2(w0.x, w0.y); wr[sx][1] = make_float2(w0.z, w0.w);
        wr[sx][2] = make_float2(w1.x, w1.y); wr[sx][3] = make_float2(w1.z, w1.w);
      }
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const uint4 raw = lds_u4(prow + (uint32_t)j * ct2);
        const uint32_t *rw = reinterpret_cast<const uint32_t *>(&raw);
        float2 xv[kV / 2];                       // bf16 -> fp32: the 16 bits moved to the top of a word
#pragma unroll
        for (int i = 0; i < 4; ++i) xv[i] = make_float2(__uint_as_float(rw[i] << 16), __uint_as_float(rw[i] & 0xFFFF0000u));
#pragma unroll
        for (int o = 0; o < TX; ++o) {
          const int sx = j - o * S;                // tap column with which input j feeds output o
          if (sx >= 0 && sx < K) {
#pragma unroll
            for (int q = 0; q < kV / 2; ++q) acc[o][q] = __ffma2_rn(xv[q], wr[sx][q], r == 0 && sx == 0 ? bz[q] : acc[o][q]);
          }
        }
      }
    }
    uint8_t *yp = reinterpret_cast<uint8_t *>(y + (((size_t)(img0 + il) * p.ho + (size_t)(y0 + ry)) * p.wo + (size_t)X0) * p.c + c0 + cv * kV);
    const int n_out = p.wo - X0;                 // outputs of this item inside the row (the last item may hang over)
#pragma unroll
    for (int o = 0; o < TX; ++o, yp += c2) {
      uint4 ov;
      uint32_t *ow = reinterpret_cast<uint32_t *>(&ov);
      // ReLU6 (compile-time): the conversion clamps at zero itself, one packed minimum against (6, 6) does
      // the rest -- the same values as clamping before rounding, since 0 and 6 are bf16 values
#pragma unroll
      for (int i = 0; i < 4; ++i)
        ow[i] = ACT ? min_bf16x2(pack_bf16x2_relu(acc[o][i].x, acc[o][i].y), 0x40C040C0u) : pack_bf16x2(acc[o][i].x, acc[o][i].y);
      if (o < n_out) *reinterpret_cast<uint4 *>(yp) = ov;
    }
    xt += d_xt;
    if (xt >= xtiles) { xt -= xtiles; ++ry; }
    ry += d_ry;
    if (ry >= rows_valid) { ry -= rows_valid; ++il; }
    il += d_il;
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

bool stencil_plan(int n, int h, int w, int c, int k, int stride, int pad, StencilParams *p) {
  if ((k != 3 && k != 5) || (stride != 1 && stride != 2) || c % kV) return false;
  const int ho = dc_out_extent(h, k, stride, pad), wo = dc_out_extent(w, k, stride, pad);
  if (ho <= 0 || wo <= 0) return false;
  p->n_img = n; p->h = h; p->w = w; p->c = c; p->ho = ho; p->wo = wo; p->pad = pad;
  // channels per tile: 32 (64-byte lines for the TMA unit; 16 measured 20 % slower, 64 leaves fewer rows per tile)
  p->ct = c % 32 == 0 ? 32 : (c % 16 == 0 ? 16 : 8);
  p->cgroups = c / p->ct;
  // patch columns: up to the last input column of the last thread item of a row (an item is tx outputs wide;
  // what lies past the image is zero-filled by the TMA unit), so that the stencil needs no column clamp
  const int tx = outputs_per_item(k, stride);
  p->in_w = (dc_div_up(wo, tx) * tx - 1) * stride + k;
  if (p->in_w > 256) return false;               // a TMA box is at most 256 elements wide
  const long long row_bytes = (long long)p->in_w * p->ct * 2;
  // rows per tile: as many as fit the patch limit, at least one
  int rt = ho;
  while (rt > 1 && ((long long)(rt - 1) * stride + k) * row_bytes > kTileBytes) --rt;
  if (((long long)(rt - 1) * stride + k) * row_bytes > kTileBytes) return false;
  if ((rt - 1) * stride + k > 256) rt = (256 - k) / stride + 1;
  p->rt = rt;
  p->ytiles = dc_div_up(ho, rt);
  p->in_rows = (rt - 1) * stride + k;
  // small maps: several images per tile while the grid still fills the GPU twice over
  p->ni = 1;
  if (p->ytiles == 1) {
    const long long img_bytes = (long long)p->in_rows * row_bytes;
    while (p->ni < 8 && p->ni * 2 <= n && (p->ni * 2) * img_bytes <= kTileBytes &&
           (long long)dc_div_up(n, p->ni * 2) * p->cgroups >= 2ll * dc_sm_count())
      p->ni *= 2;
  }
  p->igroups = dc_div_up(n, p->ni);
  p->box_bytes = (int)((long long)p->ni * p->in_rows * row_bytes);
  p->patch_bytes = (int)dc_round_up((size_t)p->box_bytes, 128);
  if ((long long)p->igroups * p->ytiles * p->cgroups >= (1ll << 31)) return false;
  return true;
}

}  // namespace

bool dc_dwconv_stencil_supported(int n, int h, int w, int c, int k, int stride, int pad) {
  StencilParams p;
  return stencil_plan(n, h, w, c, k, stride, pad, &p);
}

dc_status dc_launch_dwconv_stencil(const void *x, int n, int h, int w, int c, int k, int stride, int pad, const float *wp,
                                   const float *bias, dc_act act, void *y, cudaStream_t st) {
  StencilParams p;
  if (!stencil_plan(n, h, w, c, k, stride, pad, &p)) return DC_ERR_UNSUPPORTED;
  p.act = (int)act;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return DC_ERR_CUDA;
  CUtensorMap map_x;
  {
    const cuuint64_t C = (cuuint64_t)c;
    cuuint64_t gdim[4] = {C, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)n};
    cuuint64_t gstr[3] = {2 * C, (cuuint64_t)w * C * 2, (cuuint64_t)h * w * C * 2};
    cuuint32_t box[4] = {(cuuint32_t)p.ct, (cuuint32_t)p.in_w, (cuuint32_t)p.in_rows, (cuuint32_t)p.ni};
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = encode(&map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(x), gdim, gstr, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return DC_ERR_CUDA;
  }
  const int smem = p.patch_bytes + (k * k + 1) * p.ct * 4 + 256;
  const int grid = p.igroups * p.ytiles * p.cgroups;
  __nv_bfloat16 *yp = (__nv_bfloat16 *)y;
#define DC_DW_LAUNCH2(KK, SS, AA, CC)                                                                        \
  do {                                                                                                    \
    static unsigned char attr_done[kDcMaxDevices];                                                        \
    DC_CUDA_OK(dc_set_max_smem_once(k_dwconv_stencil<KK, SS, AA, CC>, kTileBytes + 8 * 1024, attr_done));     \
    if (dc_launch_pdl(k_dwconv_stencil<KK, SS, AA, CC>, dim3(grid), dim3(kThreads), (size_t)smem, st, map_x, p, wp, bias, yp) != cudaSuccess) \
      return DC_ERR_CUDA;                                                                                 \
  } while (0)
#define DC_DW_LAUNCH1(KK, SS, AA)                                                                         \
  do {                                                                                                    \
    if (p.ct == 32) DC_DW_LAUNCH2(KK, SS, AA, 32);                                                        \
    else DC_DW_LAUNCH2(KK, SS, AA, 0);                                                                    \
  } while (0)
#define DC_DW_LAUNCH(KK, SS)                                                                              \
  do {                                                                                                    \
    if (act == DC_ACT_RELU6) DC_DW_LAUNCH1(KK, SS, 1);                                                    \
    else DC_DW_LAUNCH1(KK, SS, 0);                                                                        \
  } while (0)
  if (k == 3 && stride == 1) DC_DW_LAUNCH(3, 1);
  else if (k == 3) DC_DW_LAUNCH(3, 2);
  else if (stride == 1) DC_DW_LAUNCH(5, 1);
  else DC_DW_LAUNCH(5, 2);
#undef DC_DW_LAUNCH2
#undef DC_DW_LAUNCH1
#undef DC_DW_LAUNCH
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}

extern "C" dc_status dc_dwconv_status(dc_stream stream) {
  DC_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  unsigned int st = 0;
  DC_CUDA_OK(cudaMemcpyFromSymbol(&st, g_dw_status, sizeof(st)));
  if (st != 0) {
    const unsigned int zero = 0;
    DC_CUDA_OK(cudaMemcpyToSymbol(g_dw_status, &zero, sizeof(zero)));
    return DC_ERR_TIMEOUT;
  }
  return DC_OK;
}
