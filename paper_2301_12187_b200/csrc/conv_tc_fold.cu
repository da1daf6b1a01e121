// Dense stride-1 convolution with few channels as an implicit GEMM whose tap COLUMNS are folded
// into the N dimension of the tensor-core instruction (see KOrder, "fold" order).
//
// Why: with 24..32 channels one tcgen05.mma of shape 128 x 32 x 16 costs the same ~48 cycles as
// one of shape 128 x 96 x 16 (it is bound by fetching the 128 x 16 activation operand from shared
// memory), so a 3x3 conv issued tap by tap is tensor-bound at 14 instructions per 128 outputs.
// Folding the k tap columns into N turns k*k*cch/2 instructions per 128 output positions into
// k*cch/2 instructions of k-fold width:
//     Z[m][s][o] = sum_{r,c} x[m + r*pitch][c] * W[o][c][r][s]          (tensor core)
//     y[m][o]    = bias[o] + sum_s Z[m + s][s][o]                       (epilogue)
// The row shift m + s of the epilogue sum is a lane shift in tensor memory: __shfl_down inside a
// warp, a small shared-memory exchange across warp boundaries, and the last k-1 rows of each
// 128-row block are recomputed by the next block (blocks advance by 128-(k-1) positions).
//
// Staging.  The operand layout is the chunk-plane scheme of conv_tc.cu: per 8-channel chunk a
// plane of all patch pixels at 16-byte pitch (the no-swizzle K-major layout), so tap row r is the
// same plane read r*pitch pixels further on.  NHWC rows do not arrive in that layout, and an SM
// pulls only ~12 bytes per cycle through per-thread 16-byte copies, so the input takes two hops:
// whole pixel rows of the patch come in by bulk copies (one per row, tracked by an mbarrier) into
// a raw ring, and the producer warps repack raw rows into chunk planes with 16-byte shared-memory
// loads and stores, writing zeros for the halo that lies outside the image.  Weights arrive once
// per CTA by one bulk copy (they are packed in HBM exactly as the operand wants them).
//
// Work split.  Tiles are th output rows of one column strip of one image, on a fixed grid; CTAs
// (one per SM) take contiguous runs of tiles and every role walks them with a few adds, no table.
// Behind the activation stages the unit is the 128-row block: blocks go round-robin over a ring of
// accumulator slots in tensor memory, the MMA warps and the epilogue groups take them in turn.
// Each epilogue warp stages its 32 rows and sends them off with its own bulk copy (the valid
// outputs of consecutive GEMM rows are contiguous in NHWC when tiles span the image width).
//
// Roles (608 threads): warps 0-2 producers, warps 3-6 MMA issue (converged warps, elected lane;
// warp 3 owns the tensor memory), warps 7-18 epilogue (three groups of four).  The kernel is bound
// by instruction issue and by the latency of the hand-offs between the roles, not by HBM or the
// tensor pipe, so waits are cheap (tight probe loops, one probing warp per epilogue group, named
// barriers elsewhere) and the per-block code is short.  All waits are bounded (tc::mbar_wait).
#include "tc_ptx.cuh"

namespace {
using namespace tc;

constexpr int kMaxRaw = 4;                       // raw row buffers (bulk copies in flight)
constexpr int kMaxStages = 4;                    // chunk-plane stages
constexpr int kMaxSlots = 6;                     // accumulator slots in tensor memory
constexpr int kProducerWarps = 3;
constexpr int kProducerThreads = kProducerWarps * 32;
constexpr int kMmaWarp = kProducerWarps;         // first MMA warp
constexpr int kMmaWarps = 4;
constexpr int kFirstEpiWarp = kMmaWarp + kMmaWarps;
constexpr int kGroups = 3;                       // epilogue groups of 4 warps
constexpr int kEpiWarps = 4 * kGroups;
constexpr int kConsumerThreads = (kMmaWarps + kEpiWarps) * 32;
constexpr int kThreads = kProducerThreads + kConsumerThreads;
constexpr int kBarConsumers = 7;                 // named barriers: 1..kGroups epilogue groups, 7 all consumers
static_assert(kGroups < kBarConsumers, "named barrier ids");
constexpr int kMaxPairs = 16;                    // tensor-core instructions per 128-row block

struct FoldParams {
  int n_img, h, w, ho, wo, c_in, c_out, co8;
  int k, pad, cch;
  int tw, th, nxt, wbox;       // tile size in outputs, x tiles per row, patch width (= GEMM row pitch)
  int tiles_y;                 // tiles per column strip
  int grid, tiles_per, tiles_rem;   // CTAs; CTA b takes tiles_per (+1 if b < tiles_rem) tiles
  int n_pad;                   // N of the instruction: k column groups of co8 channels, padded
  int blk_rows;                // output positions per 128-row block = 128 - (k-1)
  int mb, mb_last;             // blocks of a full tile / of a strip's last (shorter) tile
  int plane_stride, a_stage_bytes, b_bytes, raw_bytes;
  int nraw, stages, slots, groups, mma_warps, act, bulk_out, out_buf_bytes, xch_buf_floats;
  int off_b, off_bias, off_out, off_xch, off_raw, off_a, smem_bytes;
  int tmem_cols;
  int npairs;
  uint32_t cch_inv;            // ceil(65536 / cch): q / cch == (q * cch_inv) >> 16 for q < 4096
  uint32_t wbox_inv;           // ceil(2^20 / wbox): q / wbox == (q * wbox_inv) >> 20 for q < 4096
  uint32_t a_desc_lo[kMaxPairs];      // per instruction: (first chunk offset >> 4) | (distance >> 4) << 16
};

struct Shared {
  uint64_t raw_full[kMaxRaw], raw_empty[kMaxRaw];
  uint64_t full[kMaxStages], empty[kMaxStages];
  uint64_t slot_full[kMaxSlots], slot_empty[kMaxSlots];
  uint64_t weights;
  uint32_t tmem_base;
  uint32_t abort;
};

// Position on the tile grid; every role keeps its own and steps it once per tile.
struct Walk {
  int img, xt, ty;
  __device__ __forceinline__ void start(const FoldParams &p, int tile) {
    const int strip = tile / p.tiles_y;
    ty = tile - strip * p.tiles_y;
    img = strip / p.nxt;
    xt = strip - img * p.nxt;
  }
  __device__ __forceinline__ void step(const FoldParams &p) {
    if (++ty == p.tiles_y) {
      ty = 0;
      if (++xt == p.nxt) { xt = 0; ++img; }
    }
  }
  __device__ __forceinline__ int rows_out(const FoldParams &p) const {   // output rows of this tile
    const int left = p.ho - ty * p.th;
    return left < p.th ? left : p.th;
  }
  __device__ __forceinline__ int nblk(const FoldParams &p) const { return ty == p.tiles_y - 1 ? p.mb_last : p.mb; }
};

// Patch of a tile in image coordinates: rows [r_lo, r_hi) and columns [c_lo, c_hi) of the patch lie
// inside the image; the rest is zero padding.
struct Patch {
  int gx0, gy0, rows, r_lo, r_hi, c_lo, c_hi;
  __device__ __forceinline__ void of(const FoldParams &p, const Walk &t) {
    gx0 = t.xt * p.tw - p.pad;
    gy0 = t.ty * p.th - p.pad;
    rows = t.rows_out(p) + p.k - 1;
    r_lo = gy0 < 0 ? -gy0 : 0;
    r_hi = (p.h - gy0 < rows) ? p.h - gy0 : rows;
    c_lo = gx0 < 0 ? -gx0 : 0;
    c_hi = (p.w - gx0 < p.wbox) ? p.w - gx0 : p.wbox;
  }
};

// Epilogue of one group (4 warps = 128 threads, thread = GEMM row): blocks c = grp mod groups.
// ACT and RES are compile-time so the per-pixel code carries no runtime switches.  Per block the
// group meets at two named barriers: when the accumulator is complete (one warp watches the
// mbarrier) and when the cross-warp rows are in shared memory.  Exchange rows and staging buffers
// alternate between two copies, so a block never waits for the previous block's readers.
template <int CO8, int ACT, int RES>
__device__ __forceinline__ void epilogue_role(const FoldParams &p, Shared &sh, DcWsHeader *ws, const float *bias_s,
                                              float *xch, uint8_t *smem_out, const __nv_bfloat16 *residual,
                                              __nv_bfloat16 *y, int tile0, int ntiles) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ew = warp - kFirstEpiWarp;
  const int grp = ew >> 2;
  const int q = warp & 3;                        // tensor-memory lane quadrant this warp may read
  const bool watcher = (q == (kFirstEpiWarp & 3));
  // A waiter may trail its barrier by one phase at most, so a slot must not complete twice before
  // its group has looked: no more groups than slots take part.
  if (grp >= p.groups) return;
  const int km1 = p.k - 1;
  const int m = q * 32 + lane;
  const uint32_t tmem_row = sh.tmem_base + ((uint32_t)(q * 32) << 16);
  volatile uint32_t *abort_flag = &sh.abort;
  uint8_t *obuf0 = smem_out + (size_t)ew * 2 * p.out_buf_bytes;
  const int xch_q = (km1 * (km1 + 1) / 2) * 32;  // floats per quadrant: rows (s, lane < s), 32 channels each
  float *xg = xch + (size_t)grp * 2 * p.xch_buf_floats;
  // accumulator slot and its phase for block c = grp, advanced by the number of groups per block
  uint32_t slot = (uint32_t)grp, sph = 0;
  while (slot >= (uint32_t)p.slots) { slot -= (uint32_t)p.slots; sph ^= 1; }
  int next = grp, c0 = 0;                        // next block of this group; first block of the tile
  uint32_t mine = 0;                             // blocks this group has done
  Walk t;
  t.start(p, tile0);
#pragma unroll 1
  for (int ti = 0; ti < ntiles; ++ti) {
    const int nblk = t.nblk(p), th_t = t.rows_out(p);
    const int tw_valid = (p.wo - t.xt * p.tw < p.tw) ? p.wo - t.xt * p.tw : p.tw;
    const size_t tile_pix0 = ((size_t)t.img * p.ho + (size_t)(t.ty * p.th)) * p.wo + (size_t)(t.xt * p.tw);
#pragma unroll 1
    for (int b = next - c0; b < nblk; b += p.groups, next += p.groups) {
      bool got = true;
      if (watcher) {
        got = mbar_wait(&sh.slot_full[slot], sph, abort_flag, ws, 0x40000u | slot);
        tc_fence_before();
      }
      // the group passes or leaves together, so nobody is left alone at a named barrier
      if (!bar_all(1 + grp, 128, got)) {
        if (lane == 0) bulk_wait_all();
        return;
      }
      tc_fence_after();
      const uint32_t taddr = tmem_row + slot * (uint32_t)p.n_pad;
      float *xw = xg + (mine & 1) * p.xch_buf_floats;
      uint8_t *obuf = obuf0 + (mine & 1) * p.out_buf_bytes;
      ++mine;
      float acc[CO8];
      {
        uint32_t v[CO8];
        tmem_ld_cols<CO8>(taddr, v);
        tmem_ld_wait();
#pragma unroll
        for (int o = 0; o < CO8; o += 4) {
          const float4 bv = *reinterpret_cast<const float4 *>(bias_s + o);
          acc[o] = __uint_as_float(v[o]) + bv.x; acc[o + 1] = __uint_as_float(v[o + 1]) + bv.y;
          acc[o + 2] = __uint_as_float(v[o + 2]) + bv.z; acc[o + 3] = __uint_as_float(v[o + 3]) + bv.w;
        }
      }
#pragma unroll 1
      for (int s = 1; s <= km1; ++s) {
        uint32_t v[CO8];
        tmem_ld_cols<CO8>(taddr + (uint32_t)(s * CO8), v);
        tmem_ld_wait();
        if (lane < s) {                          // rows owed to the previous warp
          float *dst = xw + q * xch_q + ((s - 1) * s / 2 + lane) * 32;
#pragma unroll
          for (int o = 0; o < CO8; o += 4)
            *reinterpret_cast<uint4 *>(dst + o) = make_uint4(v[o], v[o + 1], v[o + 2], v[o + 3]);
        }
        const bool take = lane + s < 32;
#pragma unroll
        for (int o = 0; o < CO8; ++o) {
          const float tv = __shfl_down_sync(0xffffffffu, __uint_as_float(v[o]), s);
          if (take) acc[o] += tv;
        }
      }
      // the accumulator slot is free again: one arrival per warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.slot_empty[slot]);
      slot += (uint32_t)p.groups;
      while (slot >= (uint32_t)p.slots) { slot -= (uint32_t)p.slots; sph ^= 1; }
      bar_sync(1 + grp, 128);                    // exchange rows are visible
      if (q < 3 && lane + km1 >= 32) {
#pragma unroll 1
        for (int s = 32 - lane; s <= km1; ++s) {
          const float *src = xw + (q + 1) * xch_q + ((s - 1) * s / 2 + (lane + s - 32)) * 32;
#pragma unroll
          for (int o = 0; o < CO8; o += 4) {
            const float4 tv = *reinterpret_cast<const float4 *>(src + o);
            acc[o] += tv.x; acc[o + 1] += tv.y; acc[o + 2] += tv.z; acc[o + 3] += tv.w;
          }
        }
      }
      const int pos = b * p.blk_rows + m;
      const int yy = (int)(((uint32_t)pos * p.wbox_inv) >> 20), xx = pos - yy * p.wbox;
      const bool valid = (m < p.blk_rows) && (xx < tw_valid) && (yy < th_t);
      const int off = yy * p.wo + xx;            // pixel offset from the tile's first output pixel
      if (RES && valid) {
        const __nv_bfloat16 *rp = residual + (tile_pix0 + (size_t)off) * p.c_out;
#pragma unroll
        for (int ch = 0; ch < CO8; ch += 8) {
          if (ch < p.c_out) {
            const uint4 rv = *reinterpret_cast<const uint4 *>(rp + ch);
            const __nv_bfloat162 *rb = reinterpret_cast<const __nv_bfloat162 *>(&rv);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 rf = __bfloat1622float2(rb[i]);
              acc[ch + 2 * i] += rf.x; acc[ch + 2 * i + 1] += rf.y;
            }
          }
        }
      }
      // In lane order the valid rows of a warp are consecutive output pixels (only halo columns
      // and the tail of the block or tile drop out), so they leave as one contiguous range.
      const uint32_t vmask = __ballot_sync(0xffffffffu, valid);
      uint8_t *dst;
      if (p.bulk_out) {
        if (lane == 0) bulk_wait_read1();        // the copy that last read this buffer (two blocks ago) is done
        __syncwarp();
        dst = obuf + (size_t)__popc(vmask & ((1u << lane) - 1u)) * p.c_out * 2;
      } else {
        dst = reinterpret_cast<uint8_t *>(y + (tile_pix0 + (size_t)off) * p.c_out);
      }
      if (valid) {
#pragma unroll
        for (int ch = 0; ch < CO8; ch += 8) {
          if (ch < p.c_out) {
            uint4 ov;
            __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              float f0 = acc[ch + 2 * i], f1 = acc[ch + 2 * i + 1];
              if (ACT) { f0 = fminf(fmaxf(f0, 0.f), 6.f); f1 = fminf(fmaxf(f1, 0.f), 6.f); }
              ob[i] = __floats2bfloat162_rn(f0, f1);
            }
            *reinterpret_cast<uint4 *>(dst + ch * 2) = ov;
          }
        }
      }
      if (p.bulk_out) {
        fence_proxy_async();                     // the staged pixels are read by the bulk copy engine
        const int first = __ffs(vmask) - 1;
        const int off_first = __shfl_sync(0xffffffffu, off, first < 0 ? 0 : first);
        __syncwarp();
        if (lane == 0) {
          if (vmask)
            bulk_store(y + (tile_pix0 + (size_t)off_first) * p.c_out, smem_u32(obuf),
                       (uint32_t)(__popc(vmask) * p.c_out * 2));
          bulk_commit();                         // one group per block, empty or not: the wait above counts groups
        }
      }
    }
    c0 += nblk;
    t.step(p);
  }
  if (p.bulk_out && lane == 0) bulk_wait_all();
}

template <int CO8>
__device__ __forceinline__ void epilogue_dispatch(const FoldParams &p, Shared &sh, DcWsHeader *ws, const float *bias_s,
                                                  float *xch, uint8_t *smem_out, const __nv_bfloat16 *residual,
                                                  __nv_bfloat16 *y, int tile0, int ntiles) {
  const int v = (p.act == DC_ACT_RELU6 ? 1 : 0) | (residual ? 2 : 0);
  if (v == 0) epilogue_role<CO8, 0, 0>(p, sh, ws, bias_s, xch, smem_out, residual, y, tile0, ntiles);
  else if (v == 1) epilogue_role<CO8, 1, 0>(p, sh, ws, bias_s, xch, smem_out, residual, y, tile0, ntiles);
  else if (v == 2) epilogue_role<CO8, 0, 1>(p, sh, ws, bias_s, xch, smem_out, residual, y, tile0, ntiles);
  else epilogue_role<CO8, 1, 1>(p, sh, ws, bias_s, xch, smem_out, residual, y, tile0, ntiles);
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, const uint4 &v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
k_conv_tc_fold(const __grid_constant__ FoldParams p, const __nv_bfloat16 *__restrict__ x,
               const void *__restrict__ w_packed, const float *__restrict__ bias,
               const __nv_bfloat16 *__restrict__ residual, __nv_bfloat16 *__restrict__ y, DcWsHeader *ws) {
  extern __shared__ __align__(1024) uint8_t smem_raw_base[];
  __shared__ __align__(8) Shared sh;

  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw_base) + 1023) & ~uintptr_t(1023));
  uint8_t *smem_b = smem + p.off_b;
  uint8_t *smem_a = smem + p.off_a;
  uint8_t *smem_in = smem + p.off_raw;
  uint8_t *smem_out = smem + p.off_out;
  float *xch = reinterpret_cast<float *>(smem + p.off_xch);
  float *bias_s = reinterpret_cast<float *>(smem + p.off_bias);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile uint32_t *abort_flag = &sh.abort;

  // this CTA's run of tiles
  const int bid = (int)blockIdx.x;
  const int ntiles = p.tiles_per + (bid < p.tiles_rem ? 1 : 0);
  const int tile0 = bid * p.tiles_per + (bid < p.tiles_rem ? bid : p.tiles_rem);

  // ---- set-up: the barriers are initialised by different threads side by side
  {
    const int t = (int)threadIdx.x;
    bool did = false;
    if (t < p.nraw) { mbar_init(&sh.raw_full[t], 1); mbar_init(&sh.raw_empty[t], kProducerWarps); did = true; }
    else if (t >= 32 && t < 32 + p.stages) { mbar_init(&sh.full[t - 32], kProducerWarps); mbar_init(&sh.empty[t - 32], kMmaWarps); did = true; }
    else if (t >= 64 && t < 64 + p.slots) { mbar_init(&sh.slot_full[t - 64], 1); mbar_init(&sh.slot_empty[t - 64], 4); did = true; }
    else if (t == 95) { mbar_init(&sh.weights, 1); sh.abort = 0; did = true; }
    if (did) asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp < kProducerWarps) {
    // ================================================================== producers
    const int tid = (int)threadIdx.x;
    const int C2 = p.c_in * 2;
    const long long row_stride = (long long)p.w * C2;
    const uint32_t raw_base = smem_u32(smem_in), a_base0 = smem_u32(smem_a);
    const uint32_t raw_pitch = (uint32_t)(p.wbox * C2);
    const int row_pieces = p.wbox * p.cch;      // 16-byte pieces per patch row; piece q = (col, chunk)
    const uint32_t drow = (uint32_t)p.wbox * 16u;
    bool ok = true;

    // Warp 0 also fetches: tile j's in-image pixel rows go to raw buffer j mod nraw, one bulk copy
    // per row issued by lane (row - r_lo), all reported to the buffer's barrier.
    Walk wi;
    wi.start(p, tile0);
    int ir = 0;
    uint32_t iph = 0;
    auto fetch = [&]() {
      Patch pt;
      pt.of(p, wi);
      if (!warp_wait(&sh.raw_empty[ir], iph ^ 1, abort_flag, ws, 0x50000u | ir)) { ok = false; return; }
      const int nrows = pt.r_hi - pt.r_lo;
      const uint32_t bytes_row = (uint32_t)((pt.c_hi - pt.c_lo) * C2);
      if (lane == 0) mbar_arrive_expect_tx(&sh.raw_full[ir], (uint32_t)nrows * bytes_row);
      __syncwarp();
      if (lane < nrows) {
        const int r = pt.r_lo + lane;
        const char *src = reinterpret_cast<const char *>(x) +
                          ((long long)wi.img * p.h + (pt.gy0 + r)) * row_stride + (long long)(pt.gx0 + pt.c_lo) * C2;
        bulk_load(raw_base + (uint32_t)ir * (uint32_t)p.raw_bytes + (uint32_t)r * raw_pitch, src, bytes_row,
                  &sh.raw_full[ir]);
      }
      wi.step(p);
      if (++ir == p.nraw) { ir = 0; iph ^= 1; }
    };
    if (warp == 0) {
      if (lane == 0) {
        mbar_arrive_expect_tx(&sh.weights, (uint32_t)p.b_bytes);
        bulk_load(smem_u32(smem_b), w_packed, (uint32_t)p.b_bytes, &sh.weights);   // packed weights are the operand layout
      }
      __syncwarp();
      for (int j = 0; j < p.nraw - 1 && j < ntiles && ok; ++j) fetch();
    }

    Walk wp;
    wp.start(p, tile0);
    int s = 0, pr = 0;
    uint32_t ph = 0, pph = 0;
#pragma unroll 1
    for (int it = 0; it < ntiles && ok; ++it) {
      if (warp == 0 && it + p.nraw - 1 < ntiles) fetch();
      if (!ok) break;
      Patch pt;
      pt.of(p, wp);
      if (!mbar_wait(&sh.raw_full[pr], pph, abort_flag, ws, 0x60000u | pr)) break;
      if (!mbar_wait(&sh.empty[s], ph ^ 1, abort_flag, ws, 0x10000u | s)) break;
      const uint32_t stage = a_base0 + (uint32_t)s * (uint32_t)p.a_stage_bytes;
      const uint32_t raw = raw_base + (uint32_t)pr * (uint32_t)p.raw_bytes;
      const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 1
      for (int q = tid; q < row_pieces; q += kProducerThreads) {
        const int col = (int)(((uint32_t)q * p.cch_inv) >> 16), cc = q - col * p.cch;
        const bool cv = (col >= pt.c_lo) && (col < pt.c_hi);
        uint32_t dst = stage + (uint32_t)(cc * p.plane_stride + col * 16);
        const int lo = cv ? pt.r_lo : pt.rows, hi = cv ? pt.r_hi : pt.rows;    // rows [lo, hi) are real pixels
        int r = 0;
#pragma unroll 1
        for (; r < lo; ++r, dst += drow) sts128(dst, zero);
        uint32_t src = raw + (uint32_t)((col - pt.c_lo) * C2 + cc * 16) + (uint32_t)r * raw_pitch;
#pragma unroll 1
        for (; r + 4 <= hi; r += 4, dst += 4 * drow, src += 4 * raw_pitch) {
          const uint4 v0 = lds128(src), v1 = lds128(src + raw_pitch), v2 = lds128(src + 2 * raw_pitch),
                      v3 = lds128(src + 3 * raw_pitch);
          sts128(dst, v0); sts128(dst + drow, v1); sts128(dst + 2 * drow, v2); sts128(dst + 3 * drow, v3);
        }
#pragma unroll 1
        for (; r < hi; ++r, dst += drow, src += raw_pitch) sts128(dst, lds128(src));
#pragma unroll 1
        for (; r < pt.rows; ++r, dst += drow) sts128(dst, zero);
      }
      fence_proxy_async();                       // the planes are read by the tensor core (async proxy)
      __syncwarp();
      if (lane == 0) { mbar_arrive(&sh.full[s]); mbar_arrive(&sh.raw_empty[pr]); }
      wp.step(p);
      if (++s == p.stages) { s = 0; ph ^= 1; }
      if (++pr == p.nraw) { pr = 0; pph ^= 1; }
    }
  } else {
    // ---- consumer preparation
    if (warp == kMmaWarp) {
      tmem_alloc(&sh.tmem_base, (uint32_t)p.tmem_cols);
      tmem_relinquish();
    } else if (warp >= kFirstEpiWarp) {
      const int t = (int)threadIdx.x - kFirstEpiWarp * 32;
      if (t < 32) bias_s[t] = (bias && t < p.c_out) ? bias[t] : 0.f;
    }
    tc_fence_before();
    bar_sync(kBarConsumers, kConsumerThreads);
    tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;

    if (warp < kFirstEpiWarp) {
      // ================================================================== MMA issue
      // Warp mw takes blocks c = mw mod mma_warps.  The warps sit on different schedulers, so the
      // short issue sequences of several blocks progress side by side although each shares its
      // scheduler with busy epilogue warps.  The warp stays converged; one elected lane issues.
      const int mw = warp - kMmaWarp;
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_pad >> 3) << 17) | (8u << 24);
      const uint32_t desc_hi = (128u >> 4) | (1u << 14);
      const uint32_t b_lo0 = ((smem_u32(smem_b) >> 4) & 0x3FFFu) | ((uint32_t)p.n_pad << 16);
      const uint32_t b_step = 2u * (uint32_t)p.n_pad;
      const uint32_t a_row0 = smem_u32(smem_a) >> 4, a_stage_rows = (uint32_t)p.a_stage_bytes >> 4;
      bool ok = warp_wait(&sh.weights, 0, abort_flag, ws, 0x70000u);
      // one election for the whole role: the same lane issues a block's instructions in one stretch
      const bool leader = elect_one();
      int s = 0;                                 // stage and its phase, accumulator slot and its phase
      uint32_t ph = 0, slot = (uint32_t)mw, sph = 1, a_row = a_row0;
      while (slot >= (uint32_t)p.slots) { slot -= (uint32_t)p.slots; sph ^= 1; }
      // next block of this warp (warps beyond mma_warps take none, they only hand the stages back);
      // first block of the tile
      int next = mw < p.mma_warps ? mw : 0x40000000, c0 = 0;
      Walk t;
      t.start(p, tile0);
#pragma unroll 1
      for (int it = 0; it < ntiles && ok; ++it) {
        const int nblk = t.nblk(p);
        if (!warp_wait(&sh.full[s], ph, abort_flag, ws, 0x30000u | s)) break;
        tc_fence_after();
#pragma unroll 1
        for (int b = next - c0; b < nblk; b += p.mma_warps, next += p.mma_warps) {
          if (!warp_wait(&sh.slot_empty[slot], sph, abort_flag, ws, 0x20000u | slot)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d = tmem_base + slot * (uint32_t)p.n_pad;
          const uint32_t a_add = a_row + (uint32_t)(b * p.blk_rows);
          // statically indexed so that the table entries are read straight from the constant bank
          if (leader) {
#pragma unroll
            for (int j = 0; j < kMaxPairs; ++j) {
              if (j < p.npairs) {
                const uint64_t ad = ((uint64_t)desc_hi << 32) | (uint64_t)(p.a_desc_lo[j] + a_add);
                const uint64_t bd = ((uint64_t)desc_hi << 32) | (uint64_t)(b_lo0 + (uint32_t)j * b_step);
                umma_bf16(d, ad, bd, idesc, j != 0 ? 1u : 0u);
              }
            }
            umma_commit(&sh.slot_full[slot]);    // the block's accumulator is complete
          }
          __syncwarp();
          slot += (uint32_t)p.mma_warps;
          while (slot >= (uint32_t)p.slots) { slot -= (uint32_t)p.slots; sph ^= 1; }
        }
        // this warp's share of the stage: free once its MMAs have finished (at once if it had none)
        if (ok && leader) umma_commit(&sh.empty[s]);
        __syncwarp();
        c0 += nblk;
        t.step(p);
        a_row += a_stage_rows;
        if (++s == p.stages) { s = 0; ph ^= 1; a_row = a_row0; }
      }
    } else {
      switch (p.co8) {
        case 8: epilogue_dispatch<8>(p, sh, ws, bias_s, xch, smem_out, residual, y, tile0, ntiles); break;
        case 16: epilogue_dispatch<16>(p, sh, ws, bias_s, xch, smem_out, residual, y, tile0, ntiles); break;
        case 24: epilogue_dispatch<24>(p, sh, ws, bias_s, xch, smem_out, residual, y, tile0, ntiles); break;
        default: epilogue_dispatch<32>(p, sh, ws, bias_s, xch, smem_out, residual, y, tile0, ntiles); break;
      }
    }
    // ---- consumer teardown
    if (*abort_flag) {
      const unsigned long long t0 = globaltimer_ns();
      while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    bar_sync(kBarConsumers, kConsumerThreads);
    if (warp == kMmaWarp) {
      tc_fence_after();
      tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
  }
}

// ------------------------------------------------------------------------------------------ host
constexpr int kSmemBudget = 220 * 1024;
constexpr int kStageLimit = 40 * 1024;

// plane stride in 16-byte units, chosen so that the chunks of one pixel (written by neighbouring
// producer threads) fall into different bank groups
int padded_plane_units(int units, int cch) {
  int want = (cch == 3 || cch == 5 || cch == 7) ? cch : (cch >= 8 ? 1 : (8 / cch));
  while ((units & 7) != (want & 7)) ++units;
  return units;
}

bool fold_plan(int n, int h, int w, const dc_geom *g, int n_sm, FoldParams *p) {
  KOrder ko;
  dc_korder_init(&ko, g);
  if (!ko.fold) return false;
  const int ho = dc_out_extent(h, g->k, 1, g->pad), wo = dc_out_extent(w, g->k, 1, g->pad);
  if (ho <= 0 || wo <= 0) return false;
  if ((long long)n * h * w * g->c_in >= (1ll << 40)) return false;
  p->n_img = n; p->h = h; p->w = w; p->ho = ho; p->wo = wo;
  p->c_in = g->c_in; p->c_out = g->c_out; p->co8 = ko.co8;
  p->k = g->k; p->pad = g->pad; p->cch = ko.cch;
  p->n_pad = ko.n_pad;
  p->blk_rows = 128 - (g->k - 1);
  p->npairs = ko.e_pad / 2;
  if (p->npairs > kMaxPairs) return false;
  p->slots = 512 / p->n_pad;
  if (p->slots > kMaxSlots) p->slots = kMaxSlots;
  if (p->slots < 2) return false;
  // A waiter can trail its mbarrier by one phase at most, so every slot must have exactly one
  // MMA warp issuing into it and one epilogue group draining it: the slot count is a multiple of
  // the number of groups and of the number of MMA warps that take blocks.
  p->groups = p->slots < kGroups ? p->slots : kGroups;
  p->slots = p->slots / p->groups * p->groups;
  p->mma_warps = kMmaWarps;
  while (p->slots % p->mma_warps) --p->mma_warps;
  int cols = 32;
  while (cols < p->slots * p->n_pad) cols *= 2;
  p->tmem_cols = cols;
  p->cch_inv = (65536u + (uint32_t)p->cch - 1) / (uint32_t)p->cch;
  const int nxt = dc_div_up(wo, 64);
  p->tw = dc_div_up(wo, nxt);
  p->nxt = dc_div_up(wo, p->tw);
  p->wbox = p->tw + g->k - 1;
  if (p->wbox * p->cch >= 4096) return false;
  p->wbox_inv = ((1u << 20) + (uint32_t)p->wbox - 1) / (uint32_t)p->wbox;
  const long long strips = (long long)n * p->nxt;
  if (strips * ho >= (1ll << 30)) return false;
  const int C2 = g->c_in * 2;
  // fixed part of shared memory: weights, bias, per-warp output staging, exchange rows
  p->b_bytes = ko.e_pad * p->n_pad * 16;
  p->out_buf_bytes = (int)dc_round_up((size_t)32 * g->c_out * 2, 128);
  p->bulk_out = (p->tw == wo) ? 1 : 0;
  const int km1 = g->k - 1;
  p->xch_buf_floats = 4 * (km1 * (km1 + 1) / 2) * 32;
  const int xch_bytes = kGroups * 2 * p->xch_buf_floats * 4;
  const int slack = 4096;      // a block's 128 GEMM rows may reach past the last plane; those rows are dropped
  p->off_b = 0;
  p->off_bias = (int)dc_round_up((size_t)p->b_bytes, 128);
  p->off_out = p->off_bias + 128;
  p->off_xch = p->off_out + kEpiWarps * 2 * p->out_buf_bytes;
  p->off_raw = (int)dc_round_up((size_t)p->off_xch + xch_bytes, 128);
  auto ring_bytes = [&](int th_c, int r, int s) {
    const int rb = th_c + g->k - 1;
    const long long stage = (long long)dc_round_up((size_t)p->cch * padded_plane_units(rb * p->wbox + 1, p->cch) * 16, 128);
    const long long raw = (long long)dc_round_up((size_t)rb * p->wbox * C2, 128);
    return 1024ll + p->off_raw + r * raw + s * stage + slack;
  };
  // Rows per tile.  A CTA's time is roughly (tiles it gets) x (blocks per tile + a fixed cost per
  // tile + the patch rows it stages); the CTA with the most tiles sets the kernel's time, so the
  // candidates are ranked by that product.  Bounds: patch rows fit a warp's lanes (one bulk copy
  // per row and lane) and a stage fits its share of shared memory.
  int th = 0;
  double best = 0.0;
  for (int cand = 1; cand <= 16 && cand <= ho; ++cand) {
    const int rbox = cand + g->k - 1;
    if (rbox > 32) break;
    if ((long long)p->cch * (rbox * p->wbox + 8) * 16 > kStageLimit) break;
    if (ring_bytes(cand, 2, 2) > kSmemBudget) break;
    const long long tiles = strips * dc_div_up(ho, cand);
    const long long per_max = (tiles + n_sm - 1) / n_sm;
    const int mb = dc_div_up((cand - 1) * p->wbox + p->tw, p->blk_rows);
    double cost = (double)per_max * (mb + 0.3 + 0.05 * rbox);
    if (per_max < 3 && tiles >= 3ll * n_sm) cost *= 1.5;       // too few tiles to overlap the roles
    if (th == 0 || cost < best) { th = cand; best = cost; }
  }
  if (th == 0) return false;
  p->th = th;
  p->tiles_y = dc_div_up(ho, th);
  const long long total_tiles = strips * p->tiles_y;
  const int grid = total_tiles < n_sm ? (int)total_tiles : n_sm;
  p->grid = grid;
  p->tiles_per = (int)(total_tiles / grid);
  p->tiles_rem = (int)(total_tiles % grid);
  const int rbox = th + g->k - 1;
  p->mb = dc_div_up((th - 1) * p->wbox + p->tw, p->blk_rows);
  const int th_last = ho - (p->tiles_y - 1) * th;
  p->mb_last = dc_div_up((th_last - 1) * p->wbox + p->tw, p->blk_rows);
  p->plane_stride = padded_plane_units(rbox * p->wbox + 1, p->cch) * 16;
  p->a_stage_bytes = (int)dc_round_up((size_t)p->cch * p->plane_stride, 128);
  p->raw_bytes = (int)dc_round_up((size_t)rbox * p->wbox * C2, 128);
  // rings: as deep as the CTA's tile count and shared memory allow, the raw ring first
  const long long per_cta = p->tiles_per + (p->tiles_rem ? 1 : 0);
  int nraw = kMaxRaw < per_cta ? kMaxRaw : (int)per_cta, stages = kMaxStages < per_cta ? kMaxStages : (int)per_cta;
  if (nraw < 2) nraw = 2;
  if (stages < 2) stages = 2;
  auto total = [&](int r, int s) { return ring_bytes(th, r, s); };
  while (total(nraw, stages) > kSmemBudget && (nraw > 2 || stages > 2)) {
    if (stages >= nraw && stages > 2) --stages;
    else if (nraw > 2) --nraw;
    else --stages;
  }
  if (total(nraw, stages) > kSmemBudget) return false;
  p->nraw = nraw;
  p->stages = stages;
  p->off_a = p->off_raw + nraw * p->raw_bytes;
  p->smem_bytes = (int)total(nraw, stages);
  // chunk-pair table: entry e = (chunk cc, tap row r) -> byte offset of its 16-byte column in a stage
  for (int j = 0; j < p->npairs; ++j) {
    uint32_t off[2] = {0u, 16u};
    for (int q = 0; q < 2; ++q) {
      int pc, ccg, r, s;
      // the padding entry reads entry 0 (offset 0) again; its weights are zero
      off[q] = dc_korder_decode(ko, 2 * j + q, &pc, &ccg, &r, &s) ? (uint32_t)(ccg * p->plane_stride + r * p->wbox * 16) : 0u;
    }
    if (off[1] <= off[0]) return false;
    p->a_desc_lo[j] = (off[0] >> 4) | (((off[1] - off[0]) >> 4) << 16);
  }
  return true;
}

}  // namespace

bool dc_conv_fold_supported(int n, int h, int w, const dc_geom *g) {
  FoldParams p;
  return fold_plan(n, h, w, g, dc_sm_count(), &p);
}

dc_status dc_launch_conv_fold(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                              const float *bias, dc_act act, const void *residual, void *y, void *workspace,
                              cudaStream_t stream) {
  FoldParams p;
  const int n_sm = dc_sm_count();
  if (!fold_plan(n, h, w, g, n_sm, &p)) return DC_ERR_UNSUPPORTED;
  p.act = (int)act;
  static unsigned char attr_done[kDcMaxDevices];
  DC_CUDA_OK(dc_set_max_smem_once(k_conv_tc_fold, kSmemBudget, attr_done));
  k_conv_tc_fold<<<p.grid, kThreads, p.smem_bytes, stream>>>(p, (const __nv_bfloat16 *)x, w_packed, bias,
                                                          (const __nv_bfloat16 *)residual, (__nv_bfloat16 *)y,
                                                          (DcWsHeader *)workspace);
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}
