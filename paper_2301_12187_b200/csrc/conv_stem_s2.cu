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
// turn: one bulk copy brings a band's input rows (contiguous in memory) into one of two buffers while the
// previous band is computed, the threads widen them (four 6-byte pixels per step for three channels), one
// lane issues the band's instructions (one accumulator block per output row segment), and every
// thread reads a GEMM row back, applies the skip input and the activation and puts its pixel into an
// image of the band's output rows in shared memory, which leaves as one bulk copy (the rows are
// contiguous in memory).  With a spare fourth channel the bias rides in the weights of that channel.
// One thread waits on a barrier, the others at the CTA barrier behind it (spinning warps would take
// issue slots).  Waits are bounded.
#include "tc_ptx.cuh"

namespace {
using namespace tc;

constexpr int kThreads = 256;                    // two warps per quarter of the accumulator lanes
constexpr int kCtasPerSm = 3;
constexpr int kTmemCols = 128;                   // accumulator columns of a CTA (512 per SM)
constexpr int kSmemBudget = 73 * 1024;           // row, operand and output buffers of a CTA (three CTAs per SM)

__device__ __forceinline__ uint2 lds64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts64(uint32_t a, uint32_t x, uint32_t y) {
  asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(a), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void sts128(uint32_t a, uint4 v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

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

// PLAIN: at most three input channels (the bias rides in the weights) and no skip input; RELU: ReLU6 in
// that case (compile-time, so that the per-pixel code of the common case carries no run-time switches)
template <int PLAIN, int RELU>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
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
  uint8_t *outb = smem + p.off_stage;            // the band's output rows as they lie in memory
  const int tid = (int)threadIdx.x, warp = tid >> 5;
  volatile uint32_t *abort_flag = &abort_s;
  const int total = p.n_img * p.bands;
  // With a spare fourth channel every staged pixel carries 1.0 there, and the bias (split into two
  // bf16 terms, exact to 16 mantissa bits) sits in the weights of that channel: the tensor core adds it.
  const bool fold_bias = p.c_in <= 3;
  const uint32_t one_hi = fold_bias ? 0x3F800000u : 0u;

  // rows of band `band` of image `img` that exist in the image, as one bulk copy into row buffer `buf`
  // ([in_rows][raw_row_bytes]: rows as they are in memory)
  auto issue_load = [&](int img, int band, int buf) {
    const int Y0 = band * p.rb;
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
  // the bands of a CTA are gridDim.x apart: image and band advance by fixed steps
  const int step_img = (int)gridDim.x / p.bands, step_band = (int)gridDim.x - step_img * p.bands;
  int img = (int)blockIdx.x / p.bands, band = (int)blockIdx.x - img * p.bands;

  if (tid == 0) {
    abort_s = 0;
    mbar_init(&bar_load[0], 1);
    mbar_init(&bar_load[1], 1);
    mbar_init(&bar_mma, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Nothing above touched global memory; everything below may.  Tensor memory is allocated after this
  // point on purpose: a CTA that held columns while it waits here for the previous kernel could keep a
  // CTA of that kernel on the same SM from getting its own.
  dc_pdl_enter();
  if (tid == 0) issue_load(img, band, 0);
  if (warp == 0) {
    tmem_alloc(&tmem_base_s, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  for (int i = tid; i < p.n_pad; i += kThreads) bias_s[i] = (bias && i < p.c_out) ? bias[i] : 0.f;
  // B operand from the packed weights ([chunk plane of a tap][n_pad][8 channels]): K element (pixel s, channel c)
  // of kernel row r is W[o][c][r][s]; the fourth pixel and the spare channels carry zeros (or the bias)
  for (int i = tid; i < 3 * 4 * p.n_pad; i += kThreads) {
    const int o = i % p.n_pad, s = (i / p.n_pad) & 3, r = i / (4 * p.n_pad);
    uint2 v = make_uint2(0u, 0u);
    if (s < 3) v = *reinterpret_cast<const uint2 *>(reinterpret_cast<const uint8_t *>(w_packed) + ((size_t)(p.ent[r * 3 + s] * p.n_pad + o)) * 16);
    if (fold_bias && r == 0 && s < 2 && bias && o < p.c_out) {
      const float b = bias[o];
      const __nv_bfloat16 hi = __float2bfloat16_rn(b);
      const __nv_bfloat16 part = s == 0 ? hi : __float2bfloat16_rn(b - __bfloat162float(hi));
      v.y = (v.y & 0xFFFFu) | ((uint32_t)__bfloat16_as_ushort(part) << 16);
    }
    *reinterpret_cast<uint2 *>(bop + ((size_t)((r * 2 + (s >> 1)) * p.n_pad + o)) * 16 + (s & 1) * 8) = v;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  const uint32_t trow = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
  const bool relu6 = p.act == DC_ACT_RELU6;
  const __nv_bfloat162 zero2 = __floats2bfloat162_rn(0.f, 0.f), six2 = __floats2bfloat162_rn(6.f, 6.f);
  const int wpix = p.w + p.pad + 4;              // pixels per operand row
  const size_t out_row_bytes = (size_t)p.wo * p.c_out * 2;
  // instruction and operand descriptors (no swizzle, K-major): 128 bytes between 8-row groups; A: K chunks
  // 16 bytes apart; B: K chunks n_pad * 16 bytes apart, one descriptor per kernel row
  const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_pad >> 3) << 17) | (8u << 24);
  const uint64_t desc_hi64 = (uint64_t)((128u >> 4) | (1u << 14)) << 32;
  const uint32_t a_desc0 = smem_u32(arow) >> 4, a_row16 = (uint32_t)p.a_row_bytes >> 4;
  uint64_t b_desc[3];
#pragma unroll
  for (int r = 0; r < 3; ++r)
    b_desc[r] = desc_hi64 | (((smem_u32(bop) >> 4) + (uint32_t)(r * 2 * p.n_pad)) & 0x3FFFu) | ((uint32_t)p.n_pad << 16);

  // shared-memory addresses of the widening step, 32 bits wide (the loop below is instruction bound):
  // group j of a row = pixels 4 j .. 4 j + 3 (24 bytes) -> operand pixels 4 j + pad ..
  const uint32_t raw_s = smem_u32(smem + p.off_raw), arow_s = smem_u32(arow), out_s = smem_u32(outb);
  const int wj = tid & 63, wr0 = tid >> 6;
  const int groups = p.w >> 2;                   // w is a multiple of 8 (rows are multiples of 16 bytes)
  const uint32_t w_src0 = raw_s + (uint32_t)(wr0 * p.raw_row_bytes + wj * 24);
  const uint32_t w_dst0 = arow_s + (uint32_t)(wr0 * p.a_row_bytes + (4 * wj + p.pad) * 8);
  const uint32_t one = one_hi >> 16;
  // the pixels in front of and behind a row hold the same values in every band: written once
  for (int i = tid; i < p.in_rows * (p.pad + 4); i += kThreads) {
    const int r = i / (p.pad + 4), q = i - r * (p.pad + 4);
    const int pos = q < p.pad ? q : p.w + q;
    *reinterpret_cast<uint2 *>(arow + (size_t)r * p.a_row_bytes + pos * 8) = make_uint2(0u, one_hi);
  }

  // ---- bands of this CTA; the next band's rows arrive while this one is multiplied and written
  const int wrot = (wj >> 2) & 3;                // widen: rotation of a lane's four pixels
  const int rot = (tid >> 1) & 3;                // rotation of this lane's output pieces (read-out)
  int it = 0;
  for (int bi = (int)blockIdx.x; bi < total; bi += (int)gridDim.x, ++it) {
    const int Y0 = band * p.rb;
    const int rows_out = p.ho - Y0 < p.rb ? p.ho - Y0 : p.rb;
    const int gy0 = 2 * Y0 - p.pad;              // input row of the band's first staged row
    const int buf = it & 1;
    const int img_now = img;
    band += step_band;
    img += step_img;
    if (band >= p.bands) { band -= p.bands; ++img; }
    bool done = true;
    if (tid == 0) {
      done = mbar_wait(&bar_load[buf], (uint32_t)(it >> 1) & 1u, abort_flag, ws, 0xB0000u);
      // the other row buffer was widened one band ago: fetch the next band into it
      if (done && bi + (int)gridDim.x < total) issue_load(img, band, buf ^ 1);
    }
    tc_fence_before();                           // the previous band's accumulators have been read
    if (!__syncthreads_and(done)) break;
    // ---- widen: pixel px of staged row r goes to byte (px + pad) * 8 of its operand row; rows outside
    // the image are zeros (with 1.0 in a spare fourth channel)
    if (p.c_in == 3) {
      // four pixels (24 bytes) per step: three 8-byte loads, six byte permutes, four 8-byte stores
      uint32_t src = w_src0 + (uint32_t)(buf * p.raw_buf_bytes), dst = w_dst0;
      for (int r = wr0; r < p.in_rows; r += kThreads >> 6, src += (kThreads >> 6) * p.raw_row_bytes, dst += (kThreads >> 6) * p.a_row_bytes) {
        const bool row_in = (unsigned)(gy0 + r) < (unsigned)p.h;
        uint32_t sj = src, dj = dst;
        for (int j = wj; j < groups; j += 64, sj += 64 * 24, dj += 64 * 32) {
          uint2 a = make_uint2(0u, 0u), b = a, c = a;
          if (row_in) {
            a = lds64(sj);
            b = lds64(sj + 8);
            c = lds64(sj + 16);
          }
          // the four widened pixels leave as four 8-byte stores (the row starts `pad` pixels in, so 16-byte
          // stores would be misaligned).  A lane's 32 bytes start 32 bytes after its neighbour's: stored in the
          // same order by every lane, lanes j, j + 4, j + 8, j + 12 of a half warp would hit the same banks, so
          // lane j stores its pixel (t + j / 4) mod 4 in turn t (rotated in registers as in the read-out)
          uint2 px[4] = {make_uint2(a.x, __byte_perm(a.y, one, 0x5410)), make_uint2(__byte_perm(a.y, b.x, 0x5432), __byte_perm(b.x, one, 0x5432)),
                         make_uint2(b.y, __byte_perm(c.x, one, 0x5410)), make_uint2(__byte_perm(c.x, c.y, 0x5432), __byte_perm(c.y, one, 0x5432))};
          if (wrot & 1) { const uint2 t0 = px[0]; px[0] = px[1]; px[1] = px[2]; px[2] = px[3]; px[3] = t0; }
          if (wrot & 2) { const uint2 t0 = px[0], t1 = px[1]; px[0] = px[2]; px[1] = px[3]; px[2] = t0; px[3] = t1; }
#pragma unroll
          for (int t = 0; t < 4; ++t) sts64(dj + (uint32_t)(((t + wrot) & 3) * 8), px[t].x, px[t].y);
        }
      }
    } else {
      for (int r = tid >> 7; r < p.in_rows; r += kThreads >> 7) {
        const int gy = gy0 + r;
        const bool row_in = gy >= 0 && gy < p.h;
        const unsigned short *q0 = reinterpret_cast<const unsigned short *>(smem + p.off_raw + (size_t)buf * p.raw_buf_bytes + (size_t)r * p.raw_row_bytes);
        for (int pos = tid & 127; pos < wpix; pos += 128) {
          const int px = pos - p.pad;
          uint32_t v0 = 0u, v1 = one_hi;
          if (row_in && px >= 0 && px < p.w) {
            const unsigned short *q = q0 + px * p.c_in;
            v0 = q[0];
            if (p.c_in > 1) v0 |= (uint32_t)q[1] << 16;
            if (p.c_in > 2) v1 |= q[2];
            if (p.c_in > 3) v1 |= (uint32_t)q[3] << 16;
          }
          *reinterpret_cast<uint2 *>(arow + (size_t)r * p.a_row_bytes + pos * 8) = make_uint2(v0, v1);
        }
      }
    }
    fence_proxy_async();                         // the rows are read by the tensor core (async proxy)
    __syncthreads();
    // ---- one lane issues the band's instructions: block (row ry, segment xt) = 3 instructions
    if (warp == 0) {
      __syncwarp();
      if (elect_one()) {
        tc_fence_after();
        // output X of a segment reads 32 bytes from byte 16 X of staged row 2 ry + r (K chunks 16 bytes
        // apart); the descriptors of a band differ in the start address only
        uint32_t a_row = a_desc0;                // staged row 2 ry
        uint32_t d = tmem_base;
        for (int ry = 0; ry < rows_out; ++ry, a_row += 2 * a_row16) {
          uint32_t a_seg = a_row;
          for (int xt = 0; xt < p.xtiles; ++xt, a_seg += 128, d += (uint32_t)p.n_pad) {
            umma_bf16(d, desc_hi64 | ((a_seg) & 0x3FFFu) | (1u << 16), b_desc[0], idesc, 0u);
            umma_bf16(d, desc_hi64 | ((a_seg + a_row16) & 0x3FFFu) | (1u << 16), b_desc[1], idesc, 1u);
            umma_bf16(d, desc_hi64 | ((a_seg + 2 * a_row16) & 0x3FFFu) | (1u << 16), b_desc[2], idesc, 1u);
          }
        }
        umma_commit(&bar_mma);
      }
      __syncwarp();
    }
    if (tid == 0) {
      bulk_wait_read0();                         // the previous band's store has read the output buffer
      done = mbar_wait(&bar_mma, (uint32_t)it & 1u, abort_flag, ws, 0xB0001u);
      tc_fence_before();
    }
    if (!__syncthreads_and(done)) break;
    tc_fence_after();
    // ---- read-out: thread = GEMM row = output pixel of the segment; the two warps of a lane quarter
    // take the blocks in turn.  The band's output rows are contiguous in memory: they are put together in
    // shared memory and leave as one bulk copy.
    int blk = 0;
    for (int ry = 0; ry < rows_out; ++ry)
      for (int xt = 0; xt < p.xtiles; ++xt, ++blk) {
        if ((blk & ((kThreads >> 7) - 1)) != (warp >> 2)) continue;
        const int X = xt * 128 + (tid & 127);
        const bool valid = X < p.wo;
        const uint32_t so = out_s + (uint32_t)((ry * p.wo + X) * p.c_out * 2);
        for (int c0 = 0; c0 < p.c_out; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(trow + (uint32_t)(blk * p.n_pad + c0), v);
          tmem_ld_wait();
          if (PLAIN) {
            // A lane owns a pixel, and with 32 output channels a pixel is 64 bytes: piece g of eight neighbouring
            // lanes would fall on two 16-byte bank groups (four wavefronts per quarter warp).  Lane L therefore
            // stores its piece (t + L / 2) mod 4 in turn t: the eight lanes then hit eight different groups.  The
            // pieces are rotated in registers by two conditional moves (by one, then by two).
            uint4 ov[4];
#pragma unroll
            for (int g8 = 0; g8 < 4; ++g8) {
              uint32_t *ow = reinterpret_cast<uint32_t *>(&ov[g8]);
              // ReLU6: the conversion clamps at zero itself, one packed minimum against (6, 6) does the rest
              // (the same values as clamping before rounding, since 0 and 6 are bf16 values)
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float f0 = __uint_as_float(v[8 * g8 + 2 * i]), f1 = __uint_as_float(v[8 * g8 + 2 * i + 1]);
                ow[i] = RELU ? min_bf16x2(pack_bf16x2_relu(f0, f1), 0x40C040C0u) : pack_bf16x2(f0, f1);
              }
            }
            if (rot & 1) { const uint4 t0 = ov[0]; ov[0] = ov[1]; ov[1] = ov[2]; ov[2] = ov[3]; ov[3] = t0; }
            if (rot & 2) { const uint4 t0 = ov[0], t1 = ov[1]; ov[0] = ov[2]; ov[1] = ov[3]; ov[2] = t0; ov[3] = t1; }
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              const int g8 = (t + rot) & 3;       // the piece that now sits in ov[t]
              if (valid && c0 + 8 * g8 < p.c_out) sts128(so + (uint32_t)((c0 + 8 * g8) * 2), ov[t]);
            }
          } else {
            const size_t oi = (((size_t)img_now * p.ho + (Y0 + ry)) * p.wo + X) * p.c_out;
#pragma unroll
            for (int g8 = 0; g8 < 4; ++g8) {
              const int ch = c0 + 8 * g8;
              if (ch < p.c_out && valid) {
                float f[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[8 * g8 + i]);
                if (!fold_bias) {
#pragma unroll
                  for (int i = 0; i < 8; ++i) f[i] += bias_s[ch + i];
                }
                if (residual) {
                  const uint4 rv = *reinterpret_cast<const uint4 *>(residual + oi + ch);
                  const __nv_bfloat162 *rbp = reinterpret_cast<const __nv_bfloat162 *>(&rv);
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    const float2 rf = __bfloat1622float2(rbp[i]);
                    f[2 * i] += rf.x; f[2 * i + 1] += rf.y;
                  }
                }
                uint4 ov;
                __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  __nv_bfloat162 o2 = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
                  if (relu6) o2 = __hmin2(__hmax2(o2, zero2), six2);
                  ob[i] = o2;
                }
                sts128(so + (uint32_t)(ch * 2), ov);
              }
            }
          }
        }
      }
    fence_proxy_async();                         // the output rows are read by the bulk copy (async proxy)
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      bulk_store(reinterpret_cast<uint8_t *>(y) + ((size_t)img_now * p.ho + Y0) * out_row_bytes, out_s,
                 (uint32_t)((size_t)rows_out * out_row_bytes));
      bulk_commit();
    }
  }
  if (tid == 0) bulk_wait_all();                 // the last store has left shared memory and reached memory
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
  // output rows per CTA: accumulators within the CTA's tensor-memory columns, buffers within its share of
  // shared memory (the read-out takes 32 columns at a time, so the last block may be read past its own columns)
  const int tail = (int)dc_round_up((size_t)g->c_out, 32) - ko.n_pad;
  int rb = (kTmemCols - tail) / (p->xtiles * ko.n_pad);
  if (rb < 1) rb = 1;
  auto buffers = [&](int rows) {
    return (size_t)(2 * rows + 1) * (2 * p->raw_row_bytes + p->a_row_bytes) + (size_t)rows * wo * g->c_out * 2 +
           3 * 2 * ko.n_pad * 16 + 1024;
  };
  while (rb > 1 && buffers(rb) > kSmemBudget) --rb;
  if (buffers(rb) > kSmemBudget) return false;
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
  p->off_b = (int)dc_round_up((size_t)p->off_a + (size_t)p->in_rows * p->a_row_bytes, 128);
  p->off_stage = (int)dc_round_up((size_t)p->off_b + 3 * 2 * ko.n_pad * 16, 128);
  p->smem_bytes = p->off_stage + (int)dc_round_up((size_t)rb * wo * g->c_out * 2, 128) + 128;
  // a block's 128 GEMM rows reach 2 KB + 32 bytes into an operand row whatever the row's length: the rows
  // past the last output read what follows in shared memory (their results are not used); it must be there
  const int reach = p->off_a + p->in_rows * p->a_row_bytes + p->xtiles * 2048 + 64 + 128;
  if (p->smem_bytes < reach) p->smem_bytes = reach;
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
  // rows enter and leave by bulk copies: without 16-byte aligned images the general stem kernel runs
  if (((uintptr_t)x | (uintptr_t)y) & 15) return dc_launch_conv_stem(x, n, h, w, g, w_packed, bias, act, residual, y, workspace, stream);
  p.act = (int)act;
  const int total = n * p.bands, resident = kCtasPerSm * dc_sm_count();
  const bool plain = g->c_in <= 3 && residual == nullptr;
  cudaError_t le;
#define DC_STEM_LAUNCH(PP, RR)                                                                                      \
  do {                                                                                                              \
    static unsigned char attr_done[kDcMaxDevices];                                                                  \
    DC_CUDA_OK(dc_set_max_smem_once(k_conv_stem_s2<PP, RR>, 100 * 1024, attr_done));                                \
    le = dc_launch_pdl(k_conv_stem_s2<PP, RR>, dim3(total < resident ? total : resident), dim3(kThreads),            \
                       (size_t)p.smem_bytes, stream, p, (const __nv_bfloat16 *)x, w_packed, bias,                   \
                       (const __nv_bfloat16 *)residual, (__nv_bfloat16 *)y, (DcWsHeader *)workspace);               \
  } while (0)
  if (!plain) DC_STEM_LAUNCH(0, 0);
  else if (act == DC_ACT_RELU6) DC_STEM_LAUNCH(1, 1);
  else DC_STEM_LAUNCH(1, 0);
#undef DC_STEM_LAUNCH
  return le == cudaSuccess && cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}
