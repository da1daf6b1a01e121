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
// Staging is the chunk-plane scheme of conv_tc.cu: the haloed input patch of a tile is loaded
// once (16-byte cp.async, halo zero-filled) as planes of 8 channels at 16-byte pixel pitch, which
// is the no-swizzle K-major operand layout, so tap row r is the same plane read r*pitch pixels
// further on.  Weights arrive once per CTA by a 3-D TMA tile.
//
// The kernel is bound by the number of instructions an SM issues, so every role is written for a
// small dynamic instruction count: the CTA's tiles are decoded once into a table, loops are not
// unrolled, activation / skip-input variants are compiled separately.  Behind the activation
// stages the unit is the 128-row block: blocks go round-robin over a ring of accumulator slots in
// tensor memory, four warps issue the MMAs and three epilogue groups of four warps take the
// blocks, both in turn.  The valid outputs of a block are one contiguous range of the NHWC output when tiles
// span the image width, so each block leaves with one bulk copy.
//
// Roles (608 threads): warps 0-2 producers, warps 3-6 MMA issue (converged warps, elected lane;
// warp 3 owns the tensor memory), warps 7-18 epilogue (three groups).  Waits are bounded (tc::mbar_wait).
#include "tc_ptx.cuh"

namespace {
using namespace tc;

constexpr int kMaxStages = 8;
constexpr int kMaxSlots = 6;
constexpr int kProducerThreads = 96;
constexpr int kMmaWarp = kProducerThreads / 32;
constexpr int kGroups = 3;                       // epilogue groups of 4 warps
constexpr int kMmaWarps = 4;
constexpr int kFirstEpiWarp = kMmaWarp + kMmaWarps;
constexpr int kConsumerThreads = (kMmaWarps + 4 * kGroups) * 32;
constexpr int kThreads = kProducerThreads + kConsumerThreads;
constexpr int kBarConsumers = 7;                 // named barriers: 1..kGroups epilogue groups, 7 all consumers
static_assert(kGroups < kBarConsumers, "named barrier ids");
constexpr int kMaxTiles = 96;
constexpr int kMaxPairs = 16;                   // tensor-core instructions per 128-row block

struct FoldParams {
  int n_img, h, w, ho, wo, c_in, c_out, co8;
  int k, pad, cch;
  int tw, th, nxt, wbox;       // tile size in outputs, x tiles per row, patch width (= GEMM row pitch)
  int n_pad;                   // N of the instruction: k column groups of co8 channels, padded
  int blk_rows;                // output positions per 128-row block = 128 - (k-1)
  int mb;                      // blocks per full tile
  int total_units;             // output row segments, ordered (img, xt, y)
  int plane_stride, a_stage_bytes, b_bytes;
  int stages, slots, groups, act, bulk_out, out_buf_bytes, xch_buf_floats;
  int off_b, off_bias, off_out, off_xch, off_a, smem_bytes;
  int tmem_cols;
  int npairs;
  uint32_t cch_inv;            // ceil(65536 / cch): q / cch == (q * cch_inv) >> 16 for q < 4096
  uint32_t wbox_inv;           // ceil(2^20 / wbox): q / wbox == (q * wbox_inv) >> 20 for q < 4096
  uint32_t a_desc_lo[kMaxPairs];      // per instruction: (first chunk offset >> 4) | (distance >> 4) << 16
};

// A tile = up to p.th output rows of one column strip of one image; c0 = index of its first
// 128-row block in the CTA's block sequence.
struct Tile {
  int img, xt, y0, th, c0, nblk, rows, tw_valid;
};

struct Shared {
  uint64_t full[kMaxStages], empty[kMaxStages], slot_full[kMaxSlots], slot_empty[kMaxSlots];
  uint32_t tmem_base;
  uint32_t abort;
  int ntiles;
  Tile tiles[kMaxTiles];
};

// The CTA's contiguous range of output row segments, cut into tiles that never cross an image or
// column strip.  Written once by one thread; every role then walks the same table.
__device__ __noinline__ void build_tiles(const FoldParams &p, Shared &sh, int begin, int end) {
  int y0 = begin % p.ho;
  const int q = begin / p.ho;
  int xt = q % p.nxt, img = q / p.nxt;
  int n = 0, c = 0;
  for (int cur = begin; cur < end && n < kMaxTiles; ++n) {
    int th = p.th;
    if (th > p.ho - y0) th = p.ho - y0;
    if (th > end - cur) th = end - cur;
    Tile t;
    t.img = img; t.xt = xt; t.y0 = y0; t.th = th; t.c0 = c;
    t.rows = (th - 1) * p.wbox + p.tw;
    t.nblk = (t.rows + p.blk_rows - 1) / p.blk_rows;
    t.tw_valid = (p.wo - xt * p.tw < p.tw) ? p.wo - xt * p.tw : p.tw;
    sh.tiles[n] = t;
    c += t.nblk;
    cur += th;
    y0 += th;
    if (y0 == p.ho) { y0 = 0; if (++xt == p.nxt) { xt = 0; ++img; } }
  }
  sh.ntiles = n;
}

// Epilogue of one group (4 warps = 128 threads, thread = GEMM row): blocks c = grp mod kGroups.
// ACT and RES are compile-time so the per-pixel code carries no runtime switches.  Per block the
// group meets at two named barriers: after the cross-warp rows are in shared memory, and after the
// block's pixels are staged for the bulk copy.  Exchange rows and staging buffer alternate between
// two copies, so a block never waits for the previous block's readers.
template <int CO8, int ACT, int RES>
__device__ __forceinline__ void epilogue_role(const FoldParams &p, Shared &sh, DcWsHeader *ws, const float *bias_s,
                                              float *xch, uint8_t *smem_out, const __nv_bfloat16 *residual,
                                              __nv_bfloat16 *y) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grp = (warp - kFirstEpiWarp) >> 2;
  const int q = warp & 3;                        // tensor-memory lane quadrant this warp may read
  const bool elected = (threadIdx.x == (kFirstEpiWarp + 4 * grp) * 32);
  const int km1 = p.k - 1;
  const int m = q * 32 + lane;
  const uint32_t tmem_row = sh.tmem_base + ((uint32_t)(q * 32) << 16);
  volatile uint32_t *abort_flag = &sh.abort;
  uint8_t *obuf0 = smem_out + (size_t)grp * 2 * p.out_buf_bytes;
  const int xch_q = (km1 * (km1 + 1) / 2) * 32;  // floats per quadrant: rows (s, lane < s), 32 channels each
  float *xg = xch + (size_t)grp * 2 * p.xch_buf_floats;
  // accumulator slot and its phase for block c = grp, advanced by kGroups per block
  uint32_t slot = (uint32_t)grp, sph = 0;
  while (slot >= (uint32_t)p.slots) { slot -= (uint32_t)p.slots; sph ^= 1; }
  uint32_t next = (uint32_t)grp, mine = 0;       // next block of this group, blocks it has done
  // A waiter may trail its barrier by one phase at most, so a slot must not complete twice before
  // its group has looked: no more groups than slots take part.
  if (grp >= p.groups) return;
  const int ntiles = sh.ntiles;
#pragma unroll 1
  for (int ti = 0; ti < ntiles; ++ti) {
    const Tile t = sh.tiles[ti];
#pragma unroll 1
    for (int b = (int)next - t.c0; b < t.nblk; b += p.groups, next += p.groups) {
      // One warp watches the accumulator's barrier, the others park at the group's named barrier
      // (which costs no issue slots); the group passes or leaves together.
      bool got = true;
      if (q == (kFirstEpiWarp & 3)) {
        got = mbar_wait(&sh.slot_full[slot], sph, abort_flag, ws, 0x40000u | slot);
        tc_fence_before();
      }
      if (!bar_all(1 + grp, 128, got)) return;
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
      // the bulk copy that last read this staging buffer (two blocks ago) is done with it
      if (p.bulk_out && elected) bulk_wait_read1();
      bar_sync(1 + grp, 128);                    // exchange rows are visible, staging buffer is free
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
      const int pos0 = b * p.blk_rows;
      const int pos = pos0 + m;
      const int yy = (int)(((uint32_t)pos * p.wbox_inv) >> 20), xx = pos - yy * p.wbox;
      // first valid pixel of the block (the bulk copy starts there)
      int fy = (int)(((uint32_t)pos0 * p.wbox_inv) >> 20), fx = pos0 - fy * p.wbox;
      if (fx >= p.tw) { ++fy; fx = 0; }
      if ((m < p.blk_rows) && (xx < t.tw_valid) && (yy < t.th)) {
        const size_t pix = ((size_t)t.img * p.ho + (t.y0 + yy)) * p.wo + (t.xt * p.tw + xx);
        uint8_t *sout = obuf + (size_t)((yy - fy) * p.tw + (xx - fx)) * p.c_out * 2;
        __nv_bfloat16 *gout = y + pix * p.c_out;
#pragma unroll
        for (int ch = 0; ch < CO8; ch += 8) {
          if (ch < p.c_out) {
            if (RES) {
              const uint4 rv = *reinterpret_cast<const uint4 *>(residual + pix * p.c_out + ch);
              const __nv_bfloat162 *rb = reinterpret_cast<const __nv_bfloat162 *>(&rv);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float2 rf = __bfloat1622float2(rb[i]);
                acc[ch + 2 * i] += rf.x; acc[ch + 2 * i + 1] += rf.y;
              }
            }
            uint4 ov;
            __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              float f0 = acc[ch + 2 * i], f1 = acc[ch + 2 * i + 1];
              if (ACT) { f0 = fminf(fmaxf(f0, 0.f), 6.f); f1 = fminf(fmaxf(f1, 0.f), 6.f); }
              ob[i] = __floats2bfloat162_rn(f0, f1);
            }
            if (p.bulk_out) *reinterpret_cast<uint4 *>(sout + ch * 2) = ov;
            else *reinterpret_cast<uint4 *>(gout + ch) = ov;
          }
        }
      }
      if (p.bulk_out) {
        fence_proxy_async();                     // the staged pixels are read by the bulk copy engine
        bar_sync(1 + grp, 128);
        if (elected) {
          // the block's valid pixels are one contiguous range of the output
          int pos1 = pos0 + p.blk_rows - 1;
          if (pos1 > t.rows - 1) pos1 = t.rows - 1;
          int ly = (int)(((uint32_t)pos1 * p.wbox_inv) >> 20), lx = pos1 - ly * p.wbox;
          if (lx >= p.tw) lx = p.tw - 1;
          const int first = fy * p.tw + fx, last = ly * p.tw + lx;
          if (last >= first && fy < t.th) {
            const size_t pix0 = ((size_t)t.img * p.ho + t.y0) * p.wo + first;
            bulk_store(y + pix0 * p.c_out, smem_u32(obuf), (uint32_t)((last - first + 1) * p.c_out * 2));
          }
          bulk_commit();                         // one group per block, empty or not: the wait above counts groups
        }
      }
    }
  }
  if (p.bulk_out && elected) bulk_wait_all();
}

template <int CO8>
__device__ __forceinline__ void epilogue_dispatch(const FoldParams &p, Shared &sh, DcWsHeader *ws, const float *bias_s,
                                                  float *xch, uint8_t *smem_out, const __nv_bfloat16 *residual,
                                                  __nv_bfloat16 *y) {
  const int v = (p.act == DC_ACT_RELU6 ? 1 : 0) | (residual ? 2 : 0);
  if (v == 0) epilogue_role<CO8, 0, 0>(p, sh, ws, bias_s, xch, smem_out, residual, y);
  else if (v == 1) epilogue_role<CO8, 1, 0>(p, sh, ws, bias_s, xch, smem_out, residual, y);
  else if (v == 2) epilogue_role<CO8, 0, 1>(p, sh, ws, bias_s, xch, smem_out, residual, y);
  else epilogue_role<CO8, 1, 1>(p, sh, ws, bias_s, xch, smem_out, residual, y);
}

__global__ void __launch_bounds__(kThreads, 1)
k_conv_tc_fold(const __grid_constant__ CUtensorMap map_b, const __grid_constant__ FoldParams p,
               const __nv_bfloat16 *__restrict__ x, const float *__restrict__ bias,
               const __nv_bfloat16 *__restrict__ residual, __nv_bfloat16 *__restrict__ y, DcWsHeader *ws) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) Shared sh;

  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *smem_b = smem + p.off_b;
  uint8_t *smem_a = smem + p.off_a;
  uint8_t *smem_out = smem + p.off_out;
  float *xch = reinterpret_cast<float *>(smem + p.off_xch);
  float *bias_s = reinterpret_cast<float *>(smem + p.off_bias);

  const int warp = threadIdx.x >> 5;
  volatile uint32_t *abort_flag = &sh.abort;

  // ---- set-up.  Producers only need the barriers and the tile table, so they are released
  // first; the consumers (MMA + epilogue warps) finish their own preparation behind a second barrier.
  if (threadIdx.x == 0) {
    sh.abort = 0;
    for (int s = 0; s < p.stages; ++s) { mbar_init(&sh.full[s], kProducerThreads); mbar_init(&sh.empty[s], kMmaWarps); }
    for (int a = 0; a < p.slots; ++a) { mbar_init(&sh.slot_full[a], 1); mbar_init(&sh.slot_empty[a], 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tensormap(&map_b);
    build_tiles(p, sh, (int)((long long)p.total_units * blockIdx.x / gridDim.x),
                (int)((long long)p.total_units * (blockIdx.x + 1) / gridDim.x));
  }
  __syncthreads();
  const int ntiles = sh.ntiles;

  if (warp < kMmaWarp) {
    // ================================================================== producers
    const int ptid = threadIdx.x;
    const int row_pieces = p.wbox * p.cch;      // 16-byte pieces per patch row; piece q = (col, chunk)
    const int C2 = p.c_in * 2;
    const uint32_t a_base0 = smem_u32(smem_a);
    const long long row_stride = (long long)p.w * C2;
    const uint32_t drow_stride = (uint32_t)p.wbox * 16u;
    int s = 0;
    uint32_t ph = 0;
#pragma unroll 1
    for (int it = 0; it < ntiles; ++it) {
      const Tile t = sh.tiles[it];
      const int gx0 = t.xt * p.tw - p.pad;
      const int gy0 = t.y0 - p.pad;
      const int rows = t.th + p.k - 1;
      const int r_lo = gy0 < 0 ? -gy0 : 0;                       // patch rows [r_lo, r_hi) lie inside the image
      const int r_hi = (p.h - gy0 < rows) ? p.h - gy0 : rows;
      // pieces of a pixel row are contiguous in memory: piece q sits 16*q bytes after the row start
      const char *tile_base = reinterpret_cast<const char *>(x) + (size_t)t.img * p.h * row_stride +
                              ((long long)gy0 * p.w + gx0) * C2;
      if (!mbar_wait(&sh.empty[s], ph ^ 1, abort_flag, ws, 0x10000u | s)) break;
      if (ptid == 0 && it == 0) {
        // the weights ride on the first stage's barrier as transaction bytes and stay resident
        mbar_expect_tx(&sh.full[0], (uint32_t)p.b_bytes);
        tma_load_3d(smem_b, &map_b, &sh.full[0], 0, 0, 0);
      }
      const uint32_t stage = a_base0 + (uint32_t)s * p.a_stage_bytes;
#pragma unroll 1
      for (int q = ptid; q < row_pieces; q += kProducerThreads) {
        const int col = (int)(((uint32_t)q * p.cch_inv) >> 16), cc = q - col * p.cch;
        const int gx = gx0 + col;
        const bool cv = (gx >= 0) && (gx < p.w);
        uint32_t dst = stage + (uint32_t)(cc * p.plane_stride + col * 16);
        const int lo = cv ? r_lo : rows, hi = cv ? r_hi : rows;    // rows [lo, hi) are real pixels
        int r = 0;
#pragma unroll 1
        for (; r < lo; ++r, dst += drow_stride) cp_async16(dst, x, 0u);
        const char *src = tile_base + (long long)q * 16 + (long long)r * row_stride;
#pragma unroll 2
        for (; r < hi; ++r, dst += drow_stride, src += row_stride) cp_async16_full(dst, src);
#pragma unroll 1
        for (; r < rows; ++r, dst += drow_stride) cp_async16(dst, x, 0u);
      }
      cp_async_arrive(&sh.full[s]);              // arrives by itself when this thread's copies have landed
      if (++s == p.stages) { s = 0; ph ^= 1; }
    }
    cp_async_wait_all();                         // nothing of this thread is in flight when the CTA leaves
  } else {
    // ---- consumer preparation
    if (warp == kMmaWarp) {
      tmem_alloc(&sh.tmem_base, (uint32_t)p.tmem_cols);
      tmem_relinquish();
    } else if (warp >= kFirstEpiWarp) {
      const int t = threadIdx.x - kFirstEpiWarp * 32;
      if (t < 32) bias_s[t] = (bias && t < p.c_out) ? bias[t] : 0.f;
    }
    tc_fence_before();
    bar_sync(kBarConsumers, kConsumerThreads);
    tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;

    if (warp < kFirstEpiWarp) {
      // ================================================================== MMA issue
      // Warp mw takes blocks c = mw mod kMmaWarps.  The warps sit on different schedulers, so the
      // short issue sequences of several blocks progress side by side although each shares its
      // scheduler with busy epilogue warps.  The warp stays converged; one elected lane issues.
      const int mw = warp - kMmaWarp;
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_pad >> 3) << 17) | (8u << 24);
      const uint32_t desc_hi = (128u >> 4) | (1u << 14);
      const uint32_t b_lo0 = ((smem_u32(smem_b) >> 4) & 0x3FFFu) | ((uint32_t)p.n_pad << 16);
      const uint32_t b_step = 2u * (uint32_t)p.n_pad;
      const uint32_t a_row0 = smem_u32(smem_a) >> 4, a_stage_rows = (uint32_t)p.a_stage_bytes >> 4;
      bool ok = true;
      int s = 0;                                 // stage and its phase, accumulator slot and its phase
      uint32_t ph = 0, slot = (uint32_t)mw, sph = 1, a_row = a_row0;
      while (slot >= (uint32_t)p.slots) { slot -= (uint32_t)p.slots; sph ^= 1; }
      int next = mw;                             // next block of this warp
#pragma unroll 1
      for (int it = 0; it < ntiles && ok; ++it) {
        const int c0 = sh.tiles[it].c0, nblk = sh.tiles[it].nblk;
        if (!warp_wait(&sh.full[s], ph, abort_flag, ws, 0x30000u | s)) break;
        tc_fence_after();
#pragma unroll 1
        for (int b = next - c0; b < nblk; b += kMmaWarps, next += kMmaWarps) {
          if (!warp_wait(&sh.slot_empty[slot], sph, abort_flag, ws, 0x20000u | slot)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d = tmem_base + slot * (uint32_t)p.n_pad;
          const uint32_t a_add = a_row + (uint32_t)(b * p.blk_rows);
          // statically indexed so that the table entries are read straight from the constant bank
#pragma unroll
          for (int j = 0; j < kMaxPairs; ++j) {
            if (j < p.npairs) {
              const uint64_t ad = ((uint64_t)desc_hi << 32) | (uint64_t)(p.a_desc_lo[j] + a_add);
              const uint64_t bd = ((uint64_t)desc_hi << 32) | (uint64_t)(b_lo0 + (uint32_t)j * b_step);
              if (elect_one()) umma_bf16(d, ad, bd, idesc, j != 0 ? 1u : 0u);
            }
          }
          if (elect_one()) umma_commit(&sh.slot_full[slot]);   // the block's accumulator is complete
          slot += kMmaWarps;
          while (slot >= (uint32_t)p.slots) { slot -= (uint32_t)p.slots; sph ^= 1; }
        }
        // this warp's share of the stage: free once its MMAs have finished (at once if it had none)
        if (ok && elect_one()) umma_commit(&sh.empty[s]);
        a_row += a_stage_rows;
        if (++s == p.stages) { s = 0; ph ^= 1; a_row = a_row0; }
      }
    } else {
      switch (p.co8) {
        case 8: epilogue_dispatch<8>(p, sh, ws, bias_s, xch, smem_out, residual, y); break;
        case 16: epilogue_dispatch<16>(p, sh, ws, bias_s, xch, smem_out, residual, y); break;
        case 24: epilogue_dispatch<24>(p, sh, ws, bias_s, xch, smem_out, residual, y); break;
        default: epilogue_dispatch<32>(p, sh, ws, bias_s, xch, smem_out, residual, y); break;
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

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
}

constexpr int kSmemBudget = 220 * 1024;

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
  p->groups = p->slots < kGroups ? p->slots : kGroups;
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
  // rows per tile: bounded by the accumulator blocks, the image, shared memory, and a target of
  // about six tiles per CTA so that load, MMA and epilogue overlap
  const long long total_rows = (long long)n * ho * p->nxt;
  if (total_rows >= (1ll << 31)) return false;
  int th_target = (int)(total_rows / ((long long)n_sm * 6));
  if (th_target < 1) th_target = 1;
  int th = th_target;
  if (th > ho) th = ho;
  if (th > 16) th = 16;
  while (th > 1 && (long long)p->cch * ((th + g->k - 1) * p->wbox + 8) * 16 > 40 * 1024) --th;
  p->th = th;
  const int rbox = th + g->k - 1;
  p->mb = dc_div_up((th - 1) * p->wbox + p->tw, p->blk_rows);
  p->plane_stride = padded_plane_units(rbox * p->wbox + 1, p->cch) * 16;
  p->a_stage_bytes = (int)dc_round_up((size_t)p->cch * p->plane_stride, 128);
  p->b_bytes = ko.e_pad * p->n_pad * 16;
  p->total_units = (int)total_rows;
  // tiles of one CTA: its rows in chunks of th, plus one cut per image / column-strip boundary
  if (total_rows / n_sm / th + total_rows / n_sm / ho + 4 > kMaxTiles) return false;
  p->out_buf_bytes = (int)dc_round_up((size_t)p->blk_rows * g->c_out * 2, 128);
  p->bulk_out = (p->tw == wo) ? 1 : 0;
  const int km1 = g->k - 1;
  p->xch_buf_floats = 4 * (km1 * (km1 + 1) / 2) * 32;
  const int xch_bytes = kGroups * 2 * p->xch_buf_floats * 4;
  const int slack = p->mb * 2048 + 1024;
  p->off_b = 0;
  p->off_bias = (int)dc_round_up((size_t)p->b_bytes, 128);
  p->off_out = p->off_bias + 128;
  p->off_xch = p->off_out + kGroups * 2 * p->out_buf_bytes;
  p->off_a = (int)dc_round_up((size_t)p->off_xch + xch_bytes, 128);
  long long per_cta = total_rows / th / n_sm + 2;
  int stages = kMaxStages;
  if (stages > per_cta) stages = (int)per_cta;
  while (stages >= 2 && 1024ll + p->off_a + (long long)stages * p->a_stage_bytes + slack > kSmemBudget) --stages;
  if (stages < 2) return false;
  p->stages = stages;
  p->smem_bytes = 1024 + p->off_a + stages * p->a_stage_bytes + slack;
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
  return fold_plan(n, h, w, g, 148, &p);
}

dc_status dc_launch_conv_fold(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                              const float *bias, dc_act act, const void *residual, void *y, void *workspace,
                              cudaStream_t stream) {
  FoldParams p;
  const int n_sm = sm_count();
  if (!fold_plan(n, h, w, g, n_sm, &p)) return DC_ERR_UNSUPPORTED;
  p.act = (int)act;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return DC_ERR_CUDA;
  CUtensorMap map_b;
  {
    const int e_pad = p.npairs * 2;
    cuuint64_t gdim[3] = {8, (cuuint64_t)p.n_pad, (cuuint64_t)e_pad};
    cuuint64_t gstr[2] = {16, (cuuint64_t)p.n_pad * 16};
    cuuint32_t box[3] = {8, (cuuint32_t)p.n_pad, (cuuint32_t)e_pad};
    cuuint32_t es[3] = {1, 1, 1};
    CUresult r = encode(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(w_packed), gdim, gstr, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return DC_ERR_CUDA;
  }
  static bool attr_set = false;
  if (!attr_set) {
    DC_CUDA_OK(cudaFuncSetAttribute(k_conv_tc_fold, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
    attr_set = true;
  }
  int grid = p.total_units < n_sm ? p.total_units : n_sm;
  k_conv_tc_fold<<<grid, kThreads, p.smem_bytes, stream>>>(map_b, p, (const __nv_bfloat16 *)x, bias,
                                                          (const __nv_bfloat16 *)residual, (__nv_bfloat16 *)y,
                                                          (DcWsHeader *)workspace);
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}
