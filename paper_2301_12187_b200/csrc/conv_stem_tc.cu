// Dense convolution with very few input channels (the 3-channel stem) on the tensor core.
//
// The reduction is only k*k*c_in long and pixels are 6 bytes, so neither TMA tiles nor 16-byte
// copies can stage the operand; instead the threads build it: a CTA stages the k input rows of an
// output row segment in shared memory (coalesced 2-byte loads, zeros outside the image), then
// thread m writes, for every tap, the c_in channels of the pixel that tap reads for output m
// (padded with zeros to one 16-byte chunk) into that tap's chunk plane -- an im2col of 128 rows in
// the no-swizzle K-major layout, [tap][128 rows][16 bytes].  The packed weights are already in
// that layout ([tap][n_pad][8], general K order), so (k*k+1)/2 tcgen05.mma of shape 128 x n_pad x 16
// produce the 128 x c_out outputs of the segment in tensor memory, and each thread reads its row
// back, adds bias / skip input, applies the activation and stores 2*c_out contiguous bytes.
// Per output this is ~200 instructions instead of the ~1600 of the CUDA-core kernel (864 FMAs).
// Small CTAs (128 threads, ~35 KB of shared memory, 32..128 tensor-memory columns), several per SM,
// so staging, MMA and read-out of different segments overlap without warp specialisation.
#include "tc_ptx.cuh"

namespace {
using namespace tc;

constexpr int kStemThreads = 128;
constexpr int kStemMaxTaps = 26;                 // k <= 5: 25 taps + padding entry
constexpr int kStemVecMax = 6;                   // 16-byte chunks a thread prefetches per segment

struct StemParams {
  int n_img, h, w, ho, wo, c_in, c_out, k, stride, pad, act;
  int e_pad, n_pad, xtiles, span, tmem_cols, xrow_bytes, vec;
  unsigned nch_magic;
  int off_b, off_a, off_x, smem_bytes;
  signed char tap_r[kStemMaxTaps], tap_s[kStemMaxTaps];   // entry -> tap (r, s); -1: the zero padding entry
};

__global__ void __launch_bounds__(kStemThreads, 6)
k_conv_stem_tc(const __grid_constant__ StemParams p, const __nv_bfloat16 *__restrict__ x,
               const void *__restrict__ w_packed, const float *__restrict__ bias,
               const __nv_bfloat16 *__restrict__ residual, __nv_bfloat16 *__restrict__ y, DcWsHeader *ws) {
  extern __shared__ __align__(1024) uint8_t smem_raw_base[];
  __shared__ __align__(8) uint64_t bar_w, bar_mma;
  __shared__ uint32_t tmem_base_s, abort_s;
  __shared__ float bias_s[256];

  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw_base) + 127) & ~uintptr_t(127));
  uint8_t *smem_b = smem + p.off_b;              // [e_pad][n_pad][16 B]
  uint8_t *smem_a = smem + p.off_a;              // [e_pad][128][16 B]
  uint8_t *x_s = smem + p.off_x;                 // [k][xrow_bytes]: staged input rows
  const int tid = (int)threadIdx.x, warp = tid >> 5;
  volatile uint32_t *abort_flag = &abort_s;

  if (tid == 0) {
    abort_s = 0;
    mbar_init(&bar_w, 1);
    mbar_init(&bar_mma, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    tmem_alloc(&tmem_base_s, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  for (int i = tid; i < p.n_pad; i += kStemThreads) bias_s[i] = (bias && i < p.c_out) ? bias[i] : 0.f;
  // the padding entry's plane stays zero for the whole kernel
  for (int e = 0; e < p.e_pad; ++e)
    if (p.tap_r[e] < 0) *reinterpret_cast<uint4 *>(smem_a + ((size_t)e * 128 + tid) * 16) = make_uint4(0u, 0u, 0u, 0u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  if (tid == 0) {
    // weights: the packed layout is the operand layout, one bulk copy
    mbar_arrive_expect_tx(&bar_w, (uint32_t)(p.e_pad * p.n_pad * 16));
    bulk_load(smem_u32(smem_b), w_packed, (uint32_t)(p.e_pad * p.n_pad * 16), &bar_w);
  }
  // every wait's outcome is agreed on by the whole CTA, so that all threads leave together
  bool ok = __syncthreads_and(mbar_wait(&bar_w, 0, abort_flag, ws, 0x90000u)) != 0;

  const int row_elems = p.span * p.c_in;
  const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_pad >> 3) << 17) | (8u << 24);
  const uint32_t desc_hi = (128u >> 4) | (1u << 14);
  const uint32_t a_lo0 = ((smem_u32(smem_a) >> 4) & 0x3FFFu) | ((2048u >> 4) << 16);       // chunk planes 2 KB apart
  const uint32_t b_lo0 = ((smem_u32(smem_b) >> 4) & 0x3FFFu) | ((uint32_t)p.n_pad << 16);  // ... n_pad * 16 bytes apart
  const int nch = p.xrow_bytes >> 4, vtot = p.k * nch, rowbytes = p.w * p.c_in * 2;
  uint32_t mph = 0;
  const int total = p.n_img * p.ho * p.xtiles;   // < 2^31 (checked by the host)

  // Staging of a segment's k input rows.  With whole 16-byte chunks per image row the aligned chunks
  // covering the segment are fetched into registers (stem_fetch) and written to shared memory later
  // (stem_put), so that the fetch of the next segment overlaps this segment's MMAs and read-out.
  uint4 pre[kStemVecMax];
  auto fetch = [&](int t) {
    const int rowi = t / p.xtiles, xt = t - rowi * p.xtiles;
    const int img = rowi / p.ho, Y = rowi - img * p.ho;
    const int gy0 = Y * p.stride - p.pad;
    const int sb = (xt * 128 * p.stride - p.pad) * p.c_in * 2;
    const int ab = sb >= 0 ? (sb & ~15) : -((-sb + 15) & ~15);
    const uint8_t *xb = reinterpret_cast<const uint8_t *>(x) + (size_t)img * p.h * rowbytes;
#pragma unroll
    for (int u = 0; u < kStemVecMax; ++u) {
      const int i = u * kStemThreads + tid;
      const int r = (int)__umulhi((unsigned)i, p.nch_magic), c = i - r * nch;   // i / nch, i < 65536
      const int gy = gy0 + r;
      const int off = ab + 16 * c;
      const bool in = i < vtot && gy >= 0 && gy < p.h && off >= 0 && off + 16 <= rowbytes;
      pre[u] = in ? __ldg(reinterpret_cast<const uint4 *>(xb + (size_t)gy * rowbytes + off)) : make_uint4(0u, 0u, 0u, 0u);
    }
  };
  auto put = [&]() {
#pragma unroll
    for (int u = 0; u < kStemVecMax; ++u) {
      const int i = u * kStemThreads + tid;
      if (i < vtot) *reinterpret_cast<uint4 *>(x_s + (size_t)i * 16) = pre[u];
    }
  };
  // Image rows that are not whole chunks: 2-byte loads, batches of 8 in flight, no prefetch.
  auto stage_elems = [&](int t) {
    const int rowi = t / p.xtiles, xt = t - rowi * p.xtiles;
    const int img = rowi / p.ho, Y = rowi - img * p.ho;
    const int gy0 = Y * p.stride - p.pad;
    const int tot = p.k * row_elems, rowel = p.w * p.c_in;
    const unsigned short *xe = reinterpret_cast<const unsigned short *>(x) + (size_t)img * p.h * rowel;
    const int se = (xt * 128 * p.stride - p.pad) * p.c_in;
    for (int base = 0; base < tot; base += 8 * kStemThreads) {
      unsigned short v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = base + u * kStemThreads + tid;
        const int r = i / row_elems, c = i - r * row_elems;
        const int gy = gy0 + r;
        const int off = se + c;
        const bool in = i < tot && gy >= 0 && gy < p.h && off >= 0 && off < rowel;
        v[u] = in ? __ldg(xe + (size_t)gy * rowel + off) : (unsigned short)0;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = base + u * kStemThreads + tid;
        if (i < tot) {
          const int r = i / row_elems, c = i - r * row_elems;
          *reinterpret_cast<unsigned short *>(x_s + (size_t)r * p.xrow_bytes + 2 * c) = v[u];
        }
      }
    }
  };

  if (ok && (int)blockIdx.x < total) {
    if (p.vec) { fetch((int)blockIdx.x); put(); } else stage_elems((int)blockIdx.x);
  }
  __syncthreads();
  for (int tile = (int)blockIdx.x; tile < total && ok; tile += (int)gridDim.x) {
    const int rowi = tile / p.xtiles, xt = tile - rowi * p.xtiles;
    const int img = rowi / p.ho, Y = rowi - img * p.ho;
    const int X0 = xt * 128;
    // ---- im2col: thread = GEMM row = output pixel X0 + tid; one 16-byte chunk per tap
    {
      int shift = 0;                             // byte offset of the segment's first pixel in a staged row
      if (p.vec) {
        const int sb = (X0 * p.stride - p.pad) * p.c_in * 2;
        const int ab = sb >= 0 ? (sb & ~15) : -((-sb + 15) & ~15);
        shift = sb - ab;
      }
      const uint8_t *xp = x_s + shift + tid * p.stride * p.c_in * 2;
      for (int e = 0; e < p.e_pad; ++e) {
        const int r = p.tap_r[e], s = p.tap_s[e];
        if (r < 0) continue;
        const unsigned short *q = reinterpret_cast<const unsigned short *>(xp + r * p.xrow_bytes + s * p.c_in * 2);
        uint32_t v0 = q[0], v1 = 0u;
        if (p.c_in > 1) v0 |= (uint32_t)q[1] << 16;
        if (p.c_in > 2) v1 = q[2];
        if (p.c_in > 3) v1 |= (uint32_t)q[3] << 16;
        *reinterpret_cast<uint4 *>(smem_a + ((size_t)e * 128 + tid) * 16) = make_uint4(v0, v1, 0u, 0u);
      }
    }
    fence_proxy_async();                         // the planes are read by the tensor core (async proxy)
    tc_fence_before();
    __syncthreads();                             // planes complete; the staged rows are free again
    // ---- one thread issues the MMAs of the segment
    if (tid == 0) {
      tc_fence_after();
      for (int j = 0; j < p.e_pad / 2; ++j) {
        const uint64_t ad = ((uint64_t)desc_hi << 32) | (uint64_t)(a_lo0 + (uint32_t)j * 256u);
        const uint64_t bd = ((uint64_t)desc_hi << 32) | (uint64_t)(b_lo0 + (uint32_t)j * 2u * (uint32_t)p.n_pad);
        umma_bf16(tmem_base, ad, bd, idesc, j != 0 ? 1u : 0u);
      }
      umma_commit(&bar_mma);
    }
    const int next = tile + (int)gridDim.x;           // < 2^31 + grid: the host keeps total below 2^30
    if (p.vec && next < total) fetch(next);      // in flight during the MMAs and the read-out
    // only the issuing thread polls the mbarrier (probes cost issue slots); the others sleep at the
    // CTA barrier, and the tcgen05 fences on both sides order their tensor-memory reads after the MMAs
    bool done = true;
    if (tid == 0) {
      done = mbar_wait(&bar_mma, mph, abort_flag, ws, 0xA0000u);
      tc_fence_before();
    }
    ok = __syncthreads_and(done) != 0;
    if (!ok) break;
    mph ^= 1;
    tc_fence_after();
    // ---- read-out: thread = row; 16 columns at a time
    const int X = X0 + tid;
    const bool valid = X < p.wo;
    const size_t oi = (((size_t)img * p.ho + Y) * p.wo + X) * p.c_out;
    const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);
    for (int c0 = 0; c0 < p.c_out; c0 += 16) {
      uint32_t v[16];
      tmem_ld16(taddr + (uint32_t)c0, v);
      tmem_ld_wait();
      if (valid) {
#pragma unroll
        for (int h8 = 0; h8 < 2; ++h8) {
          const int ch = c0 + 8 * h8;
          if (ch < p.c_out) {
            float f[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[8 * h8 + i]) + bias_s[ch + i];
            if (residual) {
              const uint4 rv = *reinterpret_cast<const uint4 *>(residual + oi + ch);
              const __nv_bfloat162 *rb = reinterpret_cast<const __nv_bfloat162 *>(&rv);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float2 rf = __bfloat1622float2(rb[i]);
                f[2 * i] += rf.x; f[2 * i + 1] += rf.y;
              }
            }
            uint4 ov;
            __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              ob[i] = __floats2bfloat162_rn(dc_act_apply(f[2 * i], p.act), dc_act_apply(f[2 * i + 1], p.act));
            *reinterpret_cast<uint4 *>(y + oi + ch) = ov;
          }
        }
      }
    }
    // ---- stage the next segment's rows
    if (next < total) {
      if (p.vec) put(); else stage_elems(next);
    }
    // rows staged, accumulator read: the next segment may overwrite the planes and the accumulator
    tc_fence_before();
    __syncthreads();
  }
  if (*abort_flag) {
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

bool stem_plan(int n, int h, int w, const dc_geom *g, StemParams *p) {
  if (g->groups != 1 || g->c_in > 4 || g->c_out % 8 != 0 || g->k > 5 || g->stride > 2) return false;
  KOrder ko;
  dc_korder_init(&ko, g);
  if (ko.fold || ko.pair || ko.rows || ko.ng != 1 || ko.cch != 1) return false;
  if (ko.e_pad > kStemMaxTaps || ko.n_pad > 256) return false;
  const int ho = dc_out_extent(h, g->k, g->stride, g->pad), wo = dc_out_extent(w, g->k, g->stride, g->pad);
  if (ho <= 0 || wo <= 0) return false;
  p->n_img = n; p->h = h; p->w = w; p->ho = ho; p->wo = wo;
  p->c_in = g->c_in; p->c_out = g->c_out; p->k = g->k; p->stride = g->stride; p->pad = g->pad;
  p->e_pad = ko.e_pad; p->n_pad = ko.n_pad;
  p->xtiles = dc_div_up(wo, 128);
  if ((long long)n * ho * p->xtiles >= (1ll << 30) || (long long)w * g->c_in * 2 >= (1ll << 30)) return false;
  p->span = 127 * g->stride + g->k;
  int cols = 32;
  while (cols < ko.n_pad) cols *= 2;
  p->tmem_cols = cols;
  for (int e = 0; e < ko.e_pad; ++e) {
    int pc, ccg, r, s;
    if (dc_korder_decode(ko, e, &pc, &ccg, &r, &s)) { p->tap_r[e] = (signed char)r; p->tap_s[e] = (signed char)s; }
    else { p->tap_r[e] = -1; p->tap_s[e] = -1; }
  }
  p->off_b = 0;
  p->off_a = (int)dc_round_up((size_t)ko.e_pad * ko.n_pad * 16, 128);
  p->off_x = p->off_a + ko.e_pad * 2048;
  p->vec = (w * g->c_in) % 8 == 0;               // image rows are whole 16-byte chunks
  p->xrow_bytes = (int)dc_round_up((size_t)p->span * g->c_in * 2 + 14, 16);
  const unsigned nch = (unsigned)p->xrow_bytes / 16u;
  p->nch_magic = (unsigned)((1ull << 32) / nch) + 1u;          // (i * magic) >> 32 == i / nch for i < 65536
  if (g->k * (int)nch > kStemVecMax * kStemThreads) p->vec = 0;
  p->smem_bytes = p->off_x + g->k * p->xrow_bytes + 128;
  return p->smem_bytes <= 100 * 1024;
}

}  // namespace

bool dc_conv_stem_supported(int n, int h, int w, const dc_geom *g) {
  StemParams p;
  return stem_plan(n, h, w, g, &p);
}

dc_status dc_launch_conv_stem(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                              const float *bias, dc_act act, const void *residual, void *y, void *workspace,
                              cudaStream_t stream) {
  StemParams p;
  if (!stem_plan(n, h, w, g, &p)) return DC_ERR_UNSUPPORTED;
  p.act = (int)act;
  static unsigned char attr_done[kDcMaxDevices];
  DC_CUDA_OK(dc_set_max_smem_once(k_conv_stem_tc, 100 * 1024, attr_done));
  // several small CTAs per SM: bounded by shared memory and by 512 tensor-memory columns per SM
  int per_sm = 200 * 1024 / (p.smem_bytes + 2048);
  if (per_sm > 512 / p.tmem_cols) per_sm = 512 / p.tmem_cols;
  if (per_sm > 8) per_sm = 8;
  if (per_sm < 1) per_sm = 1;
  const long long tiles = (long long)n * p.ho * p.xtiles;
  const long long cap = (long long)dc_sm_count() * per_sm;
  const int grid = (int)(tiles < cap ? tiles : cap);
  k_conv_stem_tc<<<grid, kStemThreads, p.smem_bytes, stream>>>(p, (const __nv_bfloat16 *)x, w_packed, bias,
                                                              (const __nv_bfloat16 *)residual, (__nv_bfloat16 *)y,
                                                              (DcWsHeader *)workspace);
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}
