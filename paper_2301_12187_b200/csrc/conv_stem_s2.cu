// 3x3 stride-2 convolution with at most 4 input channels (the network's stem) on the tensor core,
// with the image rows themselves as the operand.
//
// Pixels are widened to 4 channels (8 bytes) when a row is staged in shared memory.  With stride 2
// the window of output X then starts 16 X bytes into the row (the row is stored one pixel to the right
// so that the left padding pixel is part of it), and a 32-byte K slice -- 4 pixels x 4 channels, the
// fourth pixel under zero weights -- holds all the taps of one kernel row.  Rows of the no-swizzle
// K-major operand layout are 16 bytes apart inside an 8-row group, which is exactly that window step:
// the A operand of a kernel row r is the staged image row 2Y + r - pad, read in place, with 128
// bytes between 8-row groups and 16 bytes between the two K chunks (the chunks of neighbouring
// output pixels overlap in memory).  No im2col is built: three instructions of 128 x n_pad x 16 per
// 128 outputs of an output row, and the threads only widen 6-byte pixels to 8 bytes.
//
// CTAs (256 threads, three per SM) are persistent and take bands of output rows of one image in
// turn: one bulk copy brings a band's input rows (contiguous in memory) into one of two buffers while
// the previous band is computed, the threads widen them, one lane issues the band's instructions (one
// accumulator block per output row segment), and every thread reads a GEMM row back, adds the bias /
// skip input, applies the activation and hands its pixel to the warp's turn-around buffer, from which
// four lanes write each pixel's 64-byte pieces (whole sectors).  One thread waits on a barrier, the
// others at the CTA barrier behind it (spinning warps would take issue slots).  Waits are bounded.
#include "tc_ptx.cuh"

namespace {
using namespace tc;

constexpr int kThreads = 256;                    // two warps per quarter of the accumulator lanes
constexpr int kStagePitch = 80;                  // bytes per pixel in a warp's turn-around buffer (64 + 16)

struct S2Params {
  int n_img, h, w, ho, wo, c_in, c_out, n_pad, pad, act;
  int rb, bands;               // output rows per CTA, CTAs per image
  int xtiles;                  // 128-output segments per output row
  int in_rows;                 // input rows of a band: 2 * rb + 1
  int raw_row_bytes;           // w * c_in * 2 (a multiple of 16)
  int raw_buf_bytes;           // one of the two row buffers
  int a_row_bytes;             // widened row: (w + pad + 4) pixels of 8 bytes, rounded up to 16
  int off_raw, off_a, off_b, off_stage, smem_bytes;
  int tmem_cols;
  int ent[9];                  // chunk plane of tap (r, s) in the packed weights
};

__global__ void __launch_bounds__(kThreads, 3)
k_conv_stem_s2(const __grid_constant__ S2Params p, const __nv_bfloat16 *__restrict__ x, const void *__restrict__ w_packed,
               const float *__restrict__ bias, const __nv_bfloat16 *__restrict__ residual, __nv_bfloat16 *__restrict__ y,
               DcWsHeader *ws) {
  extern __shared__ __align__(128) uint8_t smem_raw_base[];
  __shared__ __align__(8) uint64_t bar_load[2], bar_mma;
  __shared__ uint32_t tmem_base_s, abort_s;
  __shared__ float bias_s[128];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw_base) + 127) & ~uintptr_t(127));
  uint8_t *arow = smem + p.off_a;                // [in_rows][a_row_bytes]: 8-byte pixels, shifted right by pad
  uint8_t *bop = smem + p.off_b;                 // [3 kernel rows][2 K chunks][n_pad][16 bytes]
  const int tid = (int)threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile uint32_t *abort_flag = &abort_s;
  const int total = p.n_img * p.bands;

  // rows of band `bi` that exist in the image, as one bulk copy into raw buffer `buf`
  auto issue_load = [&](int bi, int buf) {
    const int img = bi / p.bands, Y0 = (bi - img * p.bands) * p.rb;
    const int rows_out = p.ho - Y0 < p.rb ? p.ho - Y0 : p.rb;
    const int gy0 = 2 * Y0 - p.pad;
    const int gy_first = gy0 < 0 ? 0 : gy0;
    int gy_last = 2 * (Y0 + rows_out - 1) - p.pad + 2;
    if (gy_last > p.h - 1) gy_last = p.h - 1;
    const uint32_t bytes = (uint32_t)((gy_last - gy_first + 1) * p.raw_row_bytes);
    mbar_arrive_expect_tx(&bar_load[buf], bytes);
    bulk_load(smem_u32(smem + p.off_raw + (size_t)buf * p.raw_buf_bytes + (size_t)(gy_first - gy0) * p.raw_row_bytes),
              reinterpret_cast<const uint8_t *>(x) + ((size_t)img * p.h + gy_first) * p.raw_row_bytes, bytes, &bar_load[buf]);
  };

  if (tid == 0) {
    abort_s = 0;
    mbar_init(&bar_load[0], 1);
    mbar_init(&bar_load[1], 1);
    mbar_init(&bar_mma, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    issue_load((int)blockIdx.x, 0);
  }
  if (warp == 0) {
    tmem_alloc(&tmem_base_s, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  for (int i = tid; i < p.n_pad; i += kThreads) bias_s[i] = (bias && i < p.c_out) ? bias[i] : 0.f;
  // B operand from the packed weights ([chunk plane of a tap][n_pad][8 channels]): K element (pixel s, channel c)
  // of kernel row r is W[o][c][r][s]; the fourth pixel and the fourth channel carry zeros
  for (int i = tid; i < 3 * 4 * p.n_pad; i += kThreads) {
    const int o = i % p.n_pad, s = (i / p.n_pad) & 3, r = i / (4 * p.n_pad);
    uint2 v = make_uint2(0u, 0u);
    if (s < 3) v = *reinterpret_cast<const uint2 *>(reinterpret_cast<const uint8_t *>(w_packed) + ((size_t)(p.ent[r * 3 + s] * p.n_pad + o)) * 16);
    *reinterpret_cast<uint2 *>(bop + ((size_t)((r * 2 + (s >> 1)) * p.n_pad + o)) * 16 + (s & 1) * 8) = v;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  uint8_t *stage = smem + p.off_stage + warp * (32 * kStagePitch);
  const uint32_t trow = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
  const bool relu6 = p.act == DC_ACT_RELU6;
  const __nv_bfloat162 zero2 = __floats2bfloat162_rn(0.f, 0.f), six2 = __floats2bfloat162_rn(6.f, 6.f);
  const int wpix = p.w + p.pad + 4;              // pixels per operand row

  // ---- bands of this CTA; the next band's rows arrive while this one is computed
  int it = 0;
  for (int bi = (int)blockIdx.x; bi < total; bi += (int)gridDim.x, ++it) {
    const int buf = it & 1;
    const int img = bi / p.bands, Y0 = (bi - img * p.bands) * p.rb;
    const int rows_out = p.ho - Y0 < p.rb ? p.ho - Y0 : p.rb;
    const int gy0 = 2 * Y0 - p.pad;              // input row of the band's first staged row
    const uint8_t *raw = smem + p.off_raw + (size_t)buf * p.raw_buf_bytes;
    bool done = true;
    if (tid == 0) {
      done = mbar_wait(&bar_load[buf], (uint32_t)(it >> 1) & 1u, abort_flag, ws, 0xB0000u);
      // the other buffer was widened one band ago; the accumulators of that band have been read
      if (done && bi + (int)gridDim.x < total) issue_load(bi + (int)gridDim.x, buf ^ 1);
    }
    tc_fence_before();
    if (!__syncthreads_and(done)) break;
    // ---- widen: pixel px of staged row r goes to byte (px + pad) * 8 of its operand row; the padding
    // pixels in front and behind, and rows outside the image, are zeros
    for (int r = tid >> 7; r < p.in_rows; r += kThreads >> 7) {
      const int gy = gy0 + r;
      const bool row_in = gy >= 0 && gy < p.h;
      const unsigned short *q0 = reinterpret_cast<const unsigned short *>(raw + (size_t)r * p.raw_row_bytes);
      for (int pos = tid & 127; pos < wpix; pos += 128) {
        const int px = pos - p.pad;
        uint32_t v0 = 0u, v1 = 0u;
        if (row_in && px >= 0 && px < p.w) {
          const unsigned short *q = q0 + px * p.c_in;
          v0 = q[0];
          if (p.c_in > 1) v0 |= (uint32_t)q[1] << 16;
          if (p.c_in > 2) v1 = q[2];
          if (p.c_in > 3) v1 |= (uint32_t)q[3] << 16;
        }
        *reinterpret_cast<uint2 *>(arow + (size_t)r * p.a_row_bytes + pos * 8) = make_uint2(v0, v1);
      }
    }
    fence_proxy_async();                         // the rows are read by the tensor core (async proxy)
    __syncthreads();
    // ---- one lane issues the band's instructions: block (row ry, segment xt) = 3 instructions
    if (warp == 0) {
      if (elect_one()) {
        tc_fence_after();
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_pad >> 3) << 17) | (8u << 24);
        const uint32_t desc_hi = (128u >> 4) | (1u << 14);     // 128 bytes between 8-row groups
        const uint32_t a_base = smem_u32(arow) >> 4, a_row16 = (uint32_t)p.a_row_bytes >> 4;
        const uint32_t b_base = ((smem_u32(bop) >> 4) & 0x3FFFu) | ((uint32_t)p.n_pad << 16);   // K chunks n_pad * 16 bytes apart
        int blk = 0;
        for (int ry = 0; ry < rows_out; ++ry)
          for (int xt = 0; xt < p.xtiles; ++xt, ++blk) {
            const uint32_t d = tmem_base + (uint32_t)(blk * p.n_pad);
#pragma unroll
            for (int r = 0; r < 3; ++r) {
              // output X of this segment reads 32 bytes from byte 16 X of staged row 2 ry + r: K chunks 16 bytes apart
              const uint32_t a_lo = ((a_base + (uint32_t)(2 * ry + r) * a_row16 + (uint32_t)(xt * 128)) & 0x3FFFu) | (1u << 16);
              const uint32_t b_lo = b_base + (uint32_t)(r * 2 * p.n_pad);
              umma_bf16(d, ((uint64_t)desc_hi << 32) | a_lo, ((uint64_t)desc_hi << 32) | b_lo, idesc, r != 0 ? 1u : 0u);
            }
          }
        umma_commit(&bar_mma);
      }
      __syncwarp();
    }
    if (tid == 0) {
      done = mbar_wait(&bar_mma, (uint32_t)it & 1u, abort_flag, ws, 0xB0001u);
      tc_fence_before();
    }
    if (!__syncthreads_and(done)) break;
    tc_fence_after();
    // ---- read-out: thread = GEMM row = output pixel of the segment; the two warps of a lane quarter
    // take the blocks in turn
    for (int blk = warp >> 2; blk < rows_out * p.xtiles; blk += kThreads >> 7) {
      const int ry = blk / p.xtiles, xt = blk - ry * p.xtiles;
      const int X = xt * 128 + (tid & 127);
      const bool valid = X < p.wo;
      const size_t oi = (((size_t)img * p.ho + (Y0 + ry)) * p.wo + X) * p.c_out;
      __nv_bfloat16 *dst = y + oi;
      const uint32_t vmask = __ballot_sync(0xffffffffu, valid);
      for (int c0 = 0; c0 < p.c_out; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(trow + (uint32_t)(blk * p.n_pad + c0), v);
        tmem_ld_wait();
#pragma unroll
        for (int g8 = 0; g8 < 4; ++g8) {
          const int ch = c0 + 8 * g8;
          uint4 ov = make_uint4(0u, 0u, 0u, 0u);
          if (ch < p.c_out) {
            float f[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[8 * g8 + i]) + bias_s[ch + i];
            if (residual && valid) {
              const uint4 rv = *reinterpret_cast<const uint4 *>(residual + oi + ch);
              const __nv_bfloat162 *rbp = reinterpret_cast<const __nv_bfloat162 *>(&rv);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float2 rf = __bfloat1622float2(rbp[i]);
                f[2 * i] += rf.x; f[2 * i + 1] += rf.y;
              }
            }
            __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              __nv_bfloat162 o2 = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
              if (relu6) o2 = __hmin2(__hmax2(o2, zero2), six2);   // same bits as clamping before rounding
              ob[i] = o2;
            }
          }
          *reinterpret_cast<uint4 *>(stage + lane * kStagePitch + g8 * 16) = ov;
        }
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int px = i * 8 + (lane >> 2), c = lane & 3;
          const unsigned long long base = __shfl_sync(0xffffffffu, (unsigned long long)(uintptr_t)dst, px);
          if (((vmask >> px) & 1u) && c0 + c * 8 < p.c_out)
            *reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>((uintptr_t)base) + c0 + c * 8) =
                *reinterpret_cast<const uint4 *>(stage + px * kStagePitch + c * 16);
        }
        __syncwarp();
      }
    }
  }
  if (*abort_flag) {                             // a copy may still be in flight: give it time to land
    const unsigned long long t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

bool s2_plan(int n, int h, int w, const dc_geom *g, S2Params *p) {
  if (g->groups != 1 || g->k != 3 || g->stride != 2 || g->pad > 1 || g->c_in > 4 || g->c_out % 8 != 0 || g->c_out > 128)
    return false;
  KOrder ko;
  dc_korder_init(&ko, g);
  if (ko.fold || ko.pair || ko.rows || ko.ng != 1 || ko.cch != 1) return false;
  const int ho = dc_out_extent(h, 3, 2, g->pad), wo = dc_out_extent(w, 3, 2, g->pad);
  if (ho <= 0 || wo <= 0) return false;
  p->n_img = n; p->h = h; p->w = w; p->ho = ho; p->wo = wo;
  p->c_in = g->c_in; p->c_out = g->c_out; p->n_pad = ko.n_pad; p->pad = g->pad;
  p->raw_row_bytes = w * g->c_in * 2;
  if (p->raw_row_bytes % 16) return false;       // rows are moved by bulk copies
  p->a_row_bytes = (int)dc_round_up((size_t)(w + g->pad + 4) * 8, 16);
  p->xtiles = dc_div_up(wo, 128);
  // the last window of a row ends at pixel 2 (wo - 1) + 3 of the operand row
  if ((2 * (wo - 1) + 4) * 8 > p->a_row_bytes) return false;
  // output rows per CTA: accumulators within 128 tensor-memory columns (four CTAs per SM), rows within ~40 KB
  // (the read-out takes 32 columns at a time, so the last block may be read past its own columns)
  const int tail = (int)dc_round_up((size_t)g->c_out, 32) - ko.n_pad;
  int rb = (128 - tail) / (p->xtiles * ko.n_pad);
  if (rb < 1) rb = 1;
  while (rb > 1 && (2 * rb + 1) * (2 * p->raw_row_bytes + p->a_row_bytes) > 44 * 1024) --rb;
  if (3 * (2 * p->raw_row_bytes + p->a_row_bytes) > 44 * 1024) return false;
  if (rb > ho) rb = ho;
  p->rb = rb;
  p->bands = dc_div_up(ho, rb);
  p->in_rows = 2 * rb + 1;
  int cols = 32;
  while (cols < rb * p->xtiles * ko.n_pad + tail) cols *= 2;
  if (cols > 256) return false;
  p->tmem_cols = cols;
  for (int r = 0; r < 3; ++r)
    for (int s = 0; s < 3; ++s) p->ent[r * 3 + s] = dc_korder_encode(ko, 0, r, s);
  p->off_raw = 0;
  p->raw_buf_bytes = (int)dc_round_up((size_t)p->in_rows * p->raw_row_bytes, 128);
  p->off_a = 2 * p->raw_buf_bytes;
  // a block's 128 GEMM rows reach 2 KB + 32 bytes into (and, in the last row, past) an operand row
  p->off_b = (int)dc_round_up((size_t)p->off_a + (size_t)p->in_rows * p->a_row_bytes + (size_t)p->xtiles * 2048 + 64, 128);
  p->off_stage = (int)dc_round_up((size_t)p->off_b + 3 * 2 * ko.n_pad * 16, 128);
  p->smem_bytes = p->off_stage + (kThreads / 32) * 32 * kStagePitch + 128;
  if ((long long)n * p->bands >= (1ll << 30)) return false;
  return p->smem_bytes <= 100 * 1024;
}

}  // namespace

bool dc_conv_stem_s2_supported(int n, int h, int w, const dc_geom *g) {
  S2Params p;
  return s2_plan(n, h, w, g, &p);
}

dc_status dc_launch_conv_stem_s2(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                                 const float *bias, dc_act act, const void *residual, void *y, void *workspace,
                                 cudaStream_t stream) {
  S2Params p;
  if (!s2_plan(n, h, w, g, &p)) return DC_ERR_UNSUPPORTED;
  p.act = (int)act;
  static unsigned char attr_done[kDcMaxDevices];
  DC_CUDA_OK(dc_set_max_smem_once(k_conv_stem_s2, 100 * 1024, attr_done));
  const int total = n * p.bands, resident = 3 * dc_sm_count();
  k_conv_stem_s2<<<total < resident ? total : resident, kThreads, p.smem_bytes, stream>>>(p, (const __nv_bfloat16 *)x, w_packed, bias,
                                                                 (const __nv_bfloat16 *)residual, (__nv_bfloat16 *)y,
                                                                 (DcWsHeader *)workspace);
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}
