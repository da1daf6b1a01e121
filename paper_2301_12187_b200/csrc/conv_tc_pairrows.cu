// Dense stride-1 convolution with few channels (c_in <= 32) as an implicit GEMM over PAIR ROWS fed
// straight from TMA tiles (see KOrder, pair == 2).
//
// A GEMM row is the 128-byte shared-memory line that holds two neighbouring input pixels, and it
// produces the two output pixels that start there:
//     D[j][e][o] = sum_{r} sum_{t} sum_{px,c} x[row y+r, pixel 2(j+t)+px][c] * W[o][c][r][2t + px - e]
// (e = 0, 1; weights are zero where 2t + px - e is no tap).  So N = 2 * c_out, the K index of a row
// is just its 16-byte chunks, tap row r and pair shift t move the operand's start address by whole
// rows, and nothing has to be rearranged between HBM and the tensor core: one 4-D TMA tile per
// patch (box = 128 bytes x pairs x rows x 1 image, 128-byte swizzle, zero fill outside the image)
// is the A operand of every instruction of the tile.  The tensor map views an image row as W/2
// pairs of 2*c_in channels; the box is 64 channels wide, so the tail of each line is zero filled.
// When the padding is odd the patch starts one pixel further left (so that pairs stay aligned in
// memory) and output pair j is (2j-1, 2j); the epilogue masks the pixel that falls off either end.
//
// Stride 2 (KOrder pair == 3) uses the same lines with ONE output per GEMM row: output X sits on
// the pixel pair it reads first, D[X][o] = sum_r sum_t sum_{px,c} x[row 2Y+r, pixel 2(X+t)+px][c] *
// W[o][c][r][2t+px-a].  Consecutive output rows need input rows two apart, so the tile is fetched as
// two TMA boxes that take every second row (even and odd patch rows); tap row r then reads box
// r & 1 from plane row r >> 1 on, and GEMM rows stay contiguous.
//
// Operand descriptors: K-major, 128-byte swizzle, 1024 bytes between 8-row groups.  Tap rows, pair
// shifts (whole 128-byte lines) and the 32-byte K step inside a line are all added to the start
// address, with the base-offset field left at 0: the tensor core applies the swizzle to the bits of
// the shared-memory address itself, exactly as the TMA engine did when it wrote the tile (stages
// are 1024-byte aligned), so any line of the tile can be row 0 of an operand.  A descriptor that
// put the start's phase, (address >> 7) & 7, into the base-offset field read wrong chunks here.
// Weights: no-swizzle K-major chunk planes, exactly as packed in HBM, one bulk copy per CTA.
//
// Work split as in the other tensor-core kernels: tiles of th output rows on a fixed grid, CTAs
// (one per SM) take contiguous runs of tiles; behind the stages the unit is the 128-row block (256
// outputs): blocks go round-robin over accumulator slots in tensor memory, the MMA warps take them
// in turn, and so do the epilogue warps, each on its own (one tensor-memory lane quadrant of every
// third block) with its own staging buffer and bulk store.
//
// Roles (512 threads): warp 0 producer (one lane issues the TMA loads), warps 1-3 MMA issue
// (converged warps, elected lane; warp 1 owns the tensor memory), warps 4-15 epilogue.  All waits
// are bounded (tc::mbar_wait).
#include "tc_ptx.cuh"

namespace {
using namespace tc;

constexpr int kMaxStages = 6;                    // activation tiles in flight
constexpr int kMaxSlots = 6;                     // accumulator slots in tensor memory
constexpr int kMmaWarp = 1;                      // first MMA warp
constexpr int kMmaWarps = 3;
constexpr int kFirstEpiWarp = kMmaWarp + kMmaWarps;
constexpr int kGroups = 3;                       // epilogue warps per tensor-memory lane quadrant
constexpr int kEpiWarps = 4 * kGroups;
constexpr int kConsumerThreads = (kMmaWarps + kEpiWarps) * 32;
constexpr int kThreads = 32 + kConsumerThreads;
constexpr int kBarConsumers = 7;                 // named barrier of all consumer warps
constexpr int kMaxMma = 64;                      // tensor-core instructions per block
constexpr int kInFlight = 3;                     // activation tiles a CTA requests ahead of their use

struct PairParams {
  int n_img, h, w, ho, wo, c_in, c_out, co8;
  int k, pad, cch;
  int stride;                  // 1: two outputs per GEMM row (a pair); 2: one output per GEMM row
  int align;                   // pad & 1: output pair j is (2j - align, 2j - align + 1) (stride 1)
  int tw, th, nxt;             // tile size in outputs, x tiles per row
  int tw2, wbox2, rbox;        // output pairs per tile row, pair rows per patch row, patch rows
  int tiles_y;                 // tiles per column strip
  int grid, tiles_per, tiles_rem;   // CTAs; CTA b takes tiles_per (+1 if b < tiles_rem) tiles
  int n_pad;                   // N of the instruction: 2 * co8, padded to 16
  int mb, mb_last;             // blocks of a full tile / of a strip's last (shorter) tile
  int a_stage_bytes, a_box_bytes, a_plane_bytes, b_bytes;   // stride 2: a stage is two planes (even / odd rows)
  int stages, slots, groups, mma_warps, act, bulk_out, out_buf_bytes;
  int off_b, off_bias, off_out, off_a, smem_bytes;
  int tmem_cols;
  int nmma;
  uint32_t wbox2_inv;          // ceil(2^20 / wbox2): q / wbox2 == (q * wbox2_inv) >> 20 for q < 4096
  uint32_t a_lo[kMaxMma];      // per instruction: byte offset of its operand in a stage, >> 4
};

struct Shared {
  uint64_t full[kMaxStages], empty[kMaxStages];
  uint64_t slot_full[kMaxSlots], slot_empty[kMaxSlots];
  uint64_t weights;
  uint32_t tmem_base;
  uint32_t abort;
};

// Position on the tile grid; every role keeps its own and steps it once per tile.
struct Walk {
  int img, xt, ty;
  __device__ __forceinline__ void start(const PairParams &p, int tile) {
    const int strip = tile / p.tiles_y;
    ty = tile - strip * p.tiles_y;
    img = strip / p.nxt;
    xt = strip - img * p.nxt;
  }
  __device__ __forceinline__ void step(const PairParams &p) {
    if (++ty == p.tiles_y) {
      ty = 0;
      if (++xt == p.nxt) { xt = 0; ++img; }
    }
  }
  __device__ __forceinline__ int rows_out(const PairParams &p) const {   // output rows of this tile
    const int left = p.ho - ty * p.th;
    return left < p.th ? left : p.th;
  }
  __device__ __forceinline__ int nblk(const PairParams &p) const { return ty == p.tiles_y - 1 ? p.mb_last : p.mb; }
};

// Epilogue of one warp: tensor-memory lane quadrant q of every block c = grp mod groups, where grp
// counts the warps of the same quadrant.  Nothing is shared with other warps: the thread of GEMM
// row m owns the two output pixels of pair m, adds the skip input (the bias is in the accumulator
// already), applies the activation, converts to bf16 and stages them; the warp's valid pixels are consecutive in the NHWC output (only
// halo pairs and the tail of the block or tile drop out), so they leave as one bulk copy.
// ACT and RES are compile-time so the per-pixel code carries no runtime switches.
template <int CO8, int ACT, int RES>
__device__ __forceinline__ void epilogue_role(const PairParams &p, Shared &sh, DcWsHeader *ws,
                                              uint8_t *smem_out, const __nv_bfloat16 *residual, __nv_bfloat16 *y,
                                              int tile0, int ntiles) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ew = warp - kFirstEpiWarp;
  const int grp = ew >> 2;
  const int q = warp & 3;                        // tensor-memory lane quadrant this warp may read
  // A waiter may trail its barrier by one phase at most, so a slot must not complete twice before
  // its warp has looked: no more warps per quadrant than slots take part.
  if (grp >= p.groups) return;
  const int m = q * 32 + lane;
  const uint32_t tmem_row = sh.tmem_base + ((uint32_t)(q * 32) << 16);
  volatile uint32_t *abort_flag = &sh.abort;
  uint8_t *obuf = smem_out + (size_t)ew * p.out_buf_bytes;
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t slot = (uint32_t)grp, sph = 0;        // accumulator slot and its phase for block c = grp
  while (slot >= (uint32_t)p.slots) { slot -= (uint32_t)p.slots; sph ^= 1; }
  int next = grp, c0 = 0;                        // next block of this warp; first block of the tile
  Walk t;
  t.start(p, tile0);
#pragma unroll 1
  for (int ti = 0; ti < ntiles; ++ti) {
    const int nblk = t.nblk(p), th_t = t.rows_out(p);
    const int tw_valid = (p.wo - t.xt * p.tw < p.tw) ? p.wo - t.xt * p.tw : p.tw;
    const size_t tile_pix0 = ((size_t)t.img * p.ho + (size_t)(t.ty * p.th)) * p.wo + (size_t)(t.xt * p.tw);
#pragma unroll 1
    for (int b = next - c0; b < nblk; b += p.groups, next += p.groups) {
      if (!warp_wait(&sh.slot_full[slot], sph, abort_flag, ws, 0x40000u | slot)) {
        if (lane == 0) bulk_wait_all();
        return;
      }
      tc_fence_after();
      const uint32_t taddr = tmem_row + slot * (uint32_t)p.n_pad;
      uint32_t v0[CO8], v1[CO8];
      tmem_ld_cols<CO8>(taddr, v0);
      if (p.stride == 1) {
        tmem_ld_cols<CO8>(taddr + (uint32_t)CO8, v1);
      } else {
#pragma unroll
        for (int i = 0; i < CO8; ++i) v1[i] = 0u;
      }
      tmem_ld_wait();
      // the accumulator slot is free again: one arrival per warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.slot_empty[slot]);
      slot += (uint32_t)p.groups;
      while (slot >= (uint32_t)p.slots) { slot -= (uint32_t)p.slots; sph ^= 1; }

      const int pos = b * 128 + m;
      const int yy = (int)(((uint32_t)pos * p.wbox2_inv) >> 20), jj = pos - yy * p.wbox2;
      // first output column of the row; -1 or >= tw_valid: no such pixel
      const int xx = p.stride == 1 ? 2 * jj - p.align : jj;
      const bool valid0 = (xx >= 0) && (xx < tw_valid) && (yy < th_t);
      const bool valid1 = (p.stride == 1) && (xx + 1 < tw_valid) && (yy < th_t);
      const int off = yy * p.wo + xx;            // pixel offset from the tile's first output pixel
      const uint32_t m0 = __ballot_sync(0xffffffffu, valid0), m1 = __ballot_sync(0xffffffffu, valid1);
      uint8_t *dst;
      if (p.bulk_out) {
        if (lane == 0) bulk_wait_read0();        // the warp's previous copy (several blocks ago) has read the buffer
        __syncwarp();
        dst = obuf + (size_t)(__popc(m0 & lt) + __popc(m1 & lt)) * p.c_out * 2;
      } else {
        dst = reinterpret_cast<uint8_t *>(y + (tile_pix0 + (size_t)off) * p.c_out);
      }
      const __nv_bfloat16 *rp = RES ? residual + (tile_pix0 + (size_t)off) * p.c_out : nullptr;
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const uint32_t *v = e ? v1 : v0;
        if (e ? valid1 : valid0) {
#pragma unroll
          for (int ch = 0; ch < CO8; ch += 8) {
            if (ch < p.c_out) {
              float f[8];                          // the bias is in the accumulator already
#pragma unroll
              for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[ch + i]);
              if (RES) {
                const uint4 rv = *reinterpret_cast<const uint4 *>(rp + e * p.c_out + ch);
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
              for (int i = 0; i < 4; ++i) {
                // ReLU6 on the rounded pair: 0 and 6 are bf16 values and rounding is monotonic, so this gives
                // the same bits as clamping before the conversion, in half the instructions
                __nv_bfloat162 o2 = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
                if (ACT) o2 = __hmin2(__hmax2(o2, __floats2bfloat162_rn(0.f, 0.f)), __floats2bfloat162_rn(6.f, 6.f));
                ob[i] = o2;
              }
              // in the staging buffer the warp's pixels are packed: the second follows the first only if there is one
              *reinterpret_cast<uint4 *>(dst + ((e && (valid0 || !p.bulk_out) ? p.c_out : 0) + ch) * 2) = ov;
            }
          }
        }
      }
      if (p.bulk_out) {
        fence_proxy_async();                     // the staged pixels are read by the bulk copy engine
        const int first = __ffs(m0 | m1) - 1;
        const int off_first = __shfl_sync(0xffffffffu, valid0 ? off : off + 1, first < 0 ? 0 : first);
        __syncwarp();
        if (lane == 0) {
          if (m0 | m1)
            bulk_store(y + (tile_pix0 + (size_t)off_first) * p.c_out, smem_u32(obuf),
                       (uint32_t)((__popc(m0) + __popc(m1)) * p.c_out * 2));
          bulk_commit();
        }
      }
    }
    c0 += nblk;
    t.step(p);
  }
  if (p.bulk_out && lane == 0) bulk_wait_all();
}

// The same for more than 32 output channels: the channels are walked 8 at a time in a run-time
// loop (any c_out that is a multiple of 8), and a thread stores its pixels' channels straight to
// global memory (2 * c_out contiguous bytes per pixel; no staging buffer of that size per warp).
__device__ __noinline__ void epilogue_wide(const PairParams &p, Shared &sh, DcWsHeader *ws,
                                           const __nv_bfloat16 *residual, __nv_bfloat16 *y, int tile0, int ntiles) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grp = (warp - kFirstEpiWarp) >> 2;
  const int q = warp & 3;
  if (grp >= p.groups) return;
  const int m = q * 32 + lane;
  const uint32_t tmem_row = sh.tmem_base + ((uint32_t)(q * 32) << 16);
  volatile uint32_t *abort_flag = &sh.abort;
  uint32_t slot = (uint32_t)grp, sph = 0;
  while (slot >= (uint32_t)p.slots) { slot -= (uint32_t)p.slots; sph ^= 1; }
  int next = grp, c0 = 0;
  Walk t;
  t.start(p, tile0);
#pragma unroll 1
  for (int ti = 0; ti < ntiles; ++ti) {
    const int nblk = t.nblk(p), th_t = t.rows_out(p);
    const int tw_valid = (p.wo - t.xt * p.tw < p.tw) ? p.wo - t.xt * p.tw : p.tw;
    const size_t tile_pix0 = ((size_t)t.img * p.ho + (size_t)(t.ty * p.th)) * p.wo + (size_t)(t.xt * p.tw);
#pragma unroll 1
    for (int b = next - c0; b < nblk; b += p.groups, next += p.groups) {
      if (!warp_wait(&sh.slot_full[slot], sph, abort_flag, ws, 0x40000u | slot)) return;
      tc_fence_after();
      const uint32_t taddr = tmem_row + slot * (uint32_t)p.n_pad;
      const int pos = b * 128 + m;
      const int yy = (int)(((uint32_t)pos * p.wbox2_inv) >> 20), jj = pos - yy * p.wbox2;
      const int xx = p.stride == 1 ? 2 * jj - p.align : jj;
      const bool valid0 = (xx >= 0) && (xx < tw_valid) && (yy < th_t);
      const bool valid1 = (p.stride == 1) && (xx + 1 < tw_valid) && (yy < th_t);
      const size_t pix = tile_pix0 + (size_t)(yy * p.wo + xx);
      __nv_bfloat16 *dst = y + pix * p.c_out;
      const __nv_bfloat16 *rp = residual ? residual + pix * p.c_out : nullptr;
#pragma unroll 1
      for (int ch = 0; ch < p.c_out; ch += 8) {
        uint32_t v0[8], v1[8];
        tmem_ld8(taddr + (uint32_t)ch, v0);
        if (p.stride == 1) {
          tmem_ld8(taddr + (uint32_t)(p.co8 + ch), v1);
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) v1[i] = 0u;
        }
        tmem_ld_wait();
        if (ch + 8 >= p.c_out) {
          // all of the accumulator has been read: the slot is free again, one arrival per warp
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.slot_empty[slot]);
        }
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const uint32_t *v = e ? v1 : v0;
          if (e ? valid1 : valid0) {
            float f[8];                            // the bias is in the accumulator already
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[i]);
            if (rp) {
              const uint4 rv = *reinterpret_cast<const uint4 *>(rp + e * p.c_out + ch);
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
            for (int i = 0; i < 4; ++i) {
              float f0 = f[2 * i], f1 = f[2 * i + 1];
              if (p.act == DC_ACT_RELU6) { f0 = fminf(fmaxf(f0, 0.f), 6.f); f1 = fminf(fmaxf(f1, 0.f), 6.f); }
              ob[i] = __floats2bfloat162_rn(f0, f1);
            }
            *reinterpret_cast<uint4 *>(dst + e * p.c_out + ch) = ov;
          }
        }
      }
      slot += (uint32_t)p.groups;
      while (slot >= (uint32_t)p.slots) { slot -= (uint32_t)p.slots; sph ^= 1; }
    }
    c0 += nblk;
    t.step(p);
  }
}

template <int CO8>
__device__ __forceinline__ void epilogue_dispatch(const PairParams &p, Shared &sh, DcWsHeader *ws,
                                                  uint8_t *smem_out, const __nv_bfloat16 *residual, __nv_bfloat16 *y,
                                                  int tile0, int ntiles) {
  const int v = (p.act == DC_ACT_RELU6 ? 1 : 0) | (residual ? 2 : 0);
  if (v == 0) epilogue_role<CO8, 0, 0>(p, sh, ws, smem_out, residual, y, tile0, ntiles);
  else if (v == 1) epilogue_role<CO8, 1, 0>(p, sh, ws, smem_out, residual, y, tile0, ntiles);
  else if (v == 2) epilogue_role<CO8, 0, 1>(p, sh, ws, smem_out, residual, y, tile0, ntiles);
  else epilogue_role<CO8, 1, 1>(p, sh, ws, smem_out, residual, y, tile0, ntiles);
}

__global__ void __launch_bounds__(kThreads, 1)
k_conv_tc_pairrows(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ PairParams p,
                   const void *__restrict__ w_packed, const float *__restrict__ bias,
                   const __nv_bfloat16 *__restrict__ residual, __nv_bfloat16 *__restrict__ y, DcWsHeader *ws) {
  extern __shared__ __align__(1024) uint8_t smem_raw_base[];
  __shared__ __align__(8) Shared sh;

  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw_base) + 1023) & ~uintptr_t(1023));
  uint8_t *smem_b = smem + p.off_b;
  uint8_t *smem_a = smem + p.off_a;              // 1024-byte aligned stages (the swizzle pattern repeats every 1024 bytes)
  uint8_t *smem_out = smem + p.off_out;
  uint8_t *smem_ones = smem + p.off_bias;        // 8 lines of the constant operand (1024-byte aligned)
  uint8_t *smem_bias = smem_ones + 1024;         // [n_pad][16 bytes]: bias as two bf16 terms, then n_pad zero rows

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
    if (t < p.stages) { mbar_init(&sh.full[t], 1); mbar_init(&sh.empty[t], kMmaWarps); did = true; }
    else if (t >= 32 && t < 32 + p.slots) { mbar_init(&sh.slot_full[t - 32], 1); mbar_init(&sh.slot_empty[t - 32], 4); did = true; }
    else if (t == 64) { mbar_init(&sh.weights, 1); sh.abort = 0; prefetch_tensormap(&map_a); did = true; }
    if (did) asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  dc_pdl_enter();                                // nothing above touched global memory; everything below may
  __syncthreads();

  if (warp == 0) {
    // ================================================================== producer
    if (lane == 0) {
      mbar_arrive_expect_tx(&sh.weights, (uint32_t)p.b_bytes);
      bulk_load(smem_u32(smem_b), w_packed, (uint32_t)p.b_bytes, &sh.weights);   // packed weights are the operand layout
      const uint32_t a_base0 = smem_u32(smem_a);
      Walk t;
      t.start(p, tile0);
      int s = 0;
      uint32_t ph = 0;
      const int inflight = p.stages < kInFlight ? p.stages : kInFlight;   // never more than there are stages
#pragma unroll 1
      for (int it = 0; it < ntiles; ++it) {
        if (!mbar_wait(&sh.empty[s], ph ^ 1, abort_flag, ws, 0x10000u | s)) break;
        // At most kInFlight tiles are on their way: every CTA starts at the same moment, and if
        // each asked for all its tiles at once the first tile (which the tensor core is waiting
        // for) would arrive together with the last.
        if (it >= inflight) {
          int sw = s - inflight;
          uint32_t pw = ph;
          if (sw < 0) { sw += p.stages; pw ^= 1; }
          if (!mbar_wait(&sh.full[sw], pw, abort_flag, ws, 0x80000u | sw)) break;
        }
        // the box always has rbox rows; rows and pairs outside the image arrive as zeros
        const uint32_t dst = a_base0 + (uint32_t)s * (uint32_t)p.a_stage_bytes;
        if (p.stride == 1) {
          mbar_arrive_expect_tx(&sh.full[s], (uint32_t)p.a_box_bytes);
          tma_load_4d(dst, &map_a, &sh.full[s], 0, (t.xt * p.tw - p.pad - p.align) >> 1, t.ty * p.th - p.pad, t.img);
        } else {
          // even and odd patch rows as two boxes (the map steps two rows at a time)
          const int px0 = t.xt * p.tw - ((p.pad + p.align) >> 1), py0 = 2 * t.ty * p.th - p.pad;
          mbar_arrive_expect_tx(&sh.full[s], 2u * (uint32_t)p.a_box_bytes);
          tma_load_4d(dst, &map_a, &sh.full[s], 0, px0, py0, t.img);
          tma_load_4d(dst + (uint32_t)p.a_plane_bytes, &map_a, &sh.full[s], 0, px0, py0 + 1, t.img);
        }
        t.step(p);
        if (++s == p.stages) { s = 0; ph ^= 1; }
      }
    }
    __syncwarp();
  } else {
    // ---- consumer preparation
    if (warp == kMmaWarp) {
      tmem_alloc(&sh.tmem_base, (uint32_t)p.tmem_cols);
      tmem_relinquish();
    } else if (warp >= kFirstEpiWarp) {
      // The bias is added by the tensor core: one instruction per block multiplies a constant operand
      // (1.0 in the first two K elements of every line) with [bias as bf16, its bf16 remainder, 0, ...]
      // per accumulator column (exact to 16 mantissa bits) before the block's other instructions
      // accumulate.  The constant operand is one 8-line group read sixteen times (group stride 0); with
      // the 128-byte swizzle the first 16-byte chunk of line r sits at chunk r.  Column n belongs to
      // output channel n mod co8 (the second pixel's columns follow the first's).
      const int t0 = (int)threadIdx.x - kFirstEpiWarp * 32;
      const int ncol = (p.stride == 1 ? 2 : 1) * p.co8;
      for (int t = t0; t < 64; t += kEpiWarps * 32)
        reinterpret_cast<uint4 *>(smem_ones)[t] = make_uint4((t & 7) == (t >> 3) ? 0x3F803F80u : 0u, 0u, 0u, 0u);
      for (int t = t0; t < 2 * p.n_pad; t += kEpiWarps * 32) {
        uint32_t w0 = 0u;
        const int ch = t < ncol ? (t >= p.co8 ? t - p.co8 : t) : p.c_out;
        if (bias && ch < p.c_out) {
          const float b = bias[ch];
          const __nv_bfloat16 hi = __float2bfloat16_rn(b);
          const __nv_bfloat16 lo = __float2bfloat16_rn(b - __bfloat162float(hi));
          w0 = (uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(lo) << 16);
        }
        reinterpret_cast<uint4 *>(smem_bias)[t] = make_uint4(w0, 0u, 0u, 0u);
      }
      fence_proxy_async();                       // both are read by the tensor core (async proxy)
    }
    tc_fence_before();
    bar_sync(kBarConsumers, kConsumerThreads);
    tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;

    if (warp < kFirstEpiWarp) {
      // ================================================================== MMA issue
      // Warp mw takes blocks c = mw mod mma_warps.  The warps sit on different schedulers, so the
      // issue sequences of several blocks progress side by side although each shares its scheduler
      // with epilogue warps.  The warp stays converged; one elected lane issues.
      const int mw = warp - kMmaWarp;
      // one election for the whole role: the warp stays converged and the same lane issues every
      // instruction (an election per instruction costs ~230 cycles, several times the instruction)
      const bool leader = elect_one();
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_pad >> 3) << 17) | (8u << 24);
      const uint32_t b_hi = (128u >> 4) | (1u << 14);            // no swizzle: 128 bytes between 8-row groups
      const uint32_t a_hi = (1024u >> 4) | (1u << 14) | (2u << 29);   // 128-byte swizzle: 1024 bytes between 8-row groups
      const uint32_t b_lo0 = ((smem_u32(smem_b) >> 4) & 0x3FFFu) | ((uint32_t)p.n_pad << 16);
      const uint32_t b_step = 2u * (uint32_t)p.n_pad;
      const uint32_t a_row0 = smem_u32(smem_a) >> 4, a_stage_rows = (uint32_t)p.a_stage_bytes >> 4;
      const uint64_t ones_desc = ((uint64_t)((1u << 14) | (2u << 29)) << 32) | (uint64_t)(((smem_u32(smem_ones) >> 4) & 0x3FFFu) | (1u << 16));
      const uint64_t bias_desc = ((uint64_t)b_hi << 32) | (uint64_t)(((smem_u32(smem_bias) >> 4) & 0x3FFFu) | ((uint32_t)p.n_pad << 16));
      bool ok = warp_wait(&sh.weights, 0, abort_flag, ws, 0x70000u);
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
          const uint32_t a_add = a_row + (uint32_t)(b * 1024);    // 128 rows of 128 bytes, in 16-byte units
          uint32_t b_lo = b_lo0;
          // one lane issues the block's instructions in one stretch (no branch per instruction)
          if (leader) {
            umma_bf16(d, ones_desc, bias_desc, idesc, 0u);               // the bias initialises the accumulator
#pragma unroll 2
            for (int j = 0; j < p.nmma; ++j, b_lo += b_step) {
              const uint64_t ad = ((uint64_t)a_hi << 32) | (uint64_t)(p.a_lo[j] + a_add);
              const uint64_t bd = ((uint64_t)b_hi << 32) | (uint64_t)b_lo;
              umma_bf16(d, ad, bd, idesc, 1u);
            }
            umma_commit(&sh.slot_full[slot]);    // the block's accumulator is complete
          }
          __syncwarp();
          slot += (uint32_t)p.mma_warps;
          while (slot >= (uint32_t)p.slots) { slot -= (uint32_t)p.slots; sph ^= 1; }
        }
        // this warp's share of the stage: free once its MMAs have finished (at once if it had none)
        if (ok && leader) umma_commit(&sh.empty[s]);
        c0 += nblk;
        t.step(p);
        a_row += a_stage_rows;
        if (++s == p.stages) { s = 0; ph ^= 1; a_row = a_row0; }
      }
    } else {
      if (p.co8 > 32) epilogue_wide(p, sh, ws, residual, y, tile0, ntiles);
      else switch (p.co8) {
        case 8: epilogue_dispatch<8>(p, sh, ws, smem_out, residual, y, tile0, ntiles); break;
        case 16: epilogue_dispatch<16>(p, sh, ws, smem_out, residual, y, tile0, ntiles); break;
        case 24: epilogue_dispatch<24>(p, sh, ws, smem_out, residual, y, tile0, ntiles); break;
        default: epilogue_dispatch<32>(p, sh, ws, smem_out, residual, y, tile0, ntiles); break;
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

constexpr int kSmemBudget = 220 * 1024;
constexpr int kStageLimit = 48 * 1024;
constexpr int kSlack = 17 * 1024;   // a block's 128 rows may reach this far past the last stage

bool pair_plan(int n, int h, int w, const dc_geom *g, int n_sm, PairParams *p) {
  KOrder ko;
  dc_korder_init(&ko, g);
  if (ko.pair != 2 && ko.pair != 3) return false;
  const int S = g->stride;
  if (w & 1) return false;                        // an image row must be a whole number of pixel pairs
  const int ho = dc_out_extent(h, g->k, S, g->pad), wo = dc_out_extent(w, g->k, S, g->pad);
  if (ho <= 0 || wo <= 0) return false;
  if ((long long)n * h * w * g->c_in >= (1ll << 40)) return false;
  p->n_img = n; p->h = h; p->w = w; p->ho = ho; p->wo = wo;
  p->c_in = g->c_in; p->c_out = g->c_out; p->co8 = ko.co8;
  p->k = g->k; p->pad = g->pad; p->cch = ko.cch;
  p->stride = S;
  p->align = g->pad & 1;
  p->n_pad = ko.n_pad;
  const int nt = ko.ns[0];
  p->nmma = g->k * nt * ko.cch;
  if (p->nmma > kMaxMma) return false;
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
  const int nxt = dc_div_up(wo, 128);
  p->tw = dc_div_up(wo, nxt);
  if (S == 1 && (p->tw & 1)) ++p->tw;            // tiles start on an even output column
  p->nxt = dc_div_up(wo, p->tw);
  p->tw2 = S == 1 ? (p->tw + p->align + 1) / 2 : p->tw;    // GEMM rows per tile row
  p->wbox2 = p->tw2 + nt - 1;
  if (p->wbox2 > 256) return false;
  p->wbox2_inv = ((1u << 20) + (uint32_t)p->wbox2 - 1) / (uint32_t)p->wbox2;
  const long long strips = (long long)n * p->nxt;
  if (strips * ho >= (1ll << 30)) return false;
  // fixed part of shared memory: weights, bias, per-warp output staging
  p->b_bytes = ko.e_pad * p->n_pad * 16;
  p->bulk_out = (p->nxt == 1 && ko.co8 <= 32) ? 1 : 0;     // wider outputs are stored straight from registers
  p->out_buf_bytes = p->bulk_out ? (int)dc_round_up((size_t)(S == 1 ? 64 : 32) * g->c_out * 2, 128) : 0;
  p->off_b = 0;
  p->off_bias = (int)dc_round_up((size_t)p->b_bytes, 1024);                       // constant operand, bias rows, zero rows
  p->off_a = (int)dc_round_up((size_t)p->off_bias + 1024 + 2 * (size_t)p->n_pad * 16, 1024);
  // the output staging buffers follow the stages and double as the room a block's last rows may
  // reach into past the last stage (what is read there only feeds rows that are dropped)
  const long long tail_bytes = kEpiWarps * p->out_buf_bytes > kSlack ? kEpiWarps * p->out_buf_bytes : kSlack;
  // patch rows of a tile of th_c output rows; stride 2 holds them as two planes of every second row
  auto patch_rows = [&](int th_c) { return S == 1 ? th_c + g->k - 1 : 2 * (th_c - 1) + g->k; };
  auto plane_bytes = [&](int th_c) {
    const int rows = S == 1 ? patch_rows(th_c) : (patch_rows(th_c) + 1) / 2;
    return (long long)dc_round_up((size_t)rows * p->wbox2 * 128, 1024);
  };
  auto stage_bytes = [&](int th_c) { return S * plane_bytes(th_c); };
  auto total_bytes = [&](int th_c, int s) { return 1024ll + p->off_a + s * stage_bytes(th_c) + tail_bytes; };
  // Rows per tile.  A CTA's time is roughly (tiles it gets) x (blocks per tile + a fixed cost per
  // tile + the patch rows it stages) plus the start-up of its first tile, which nothing overlaps;
  // the CTA with the most tiles sets the kernel's time, so the candidates are ranked by that sum.
  int th = 0;
  double best = 0.0;
  for (int cand = 1; cand <= 32 && cand <= ho; ++cand) {
    const int rbox = patch_rows(cand);
    if (rbox > 127) break;
    if (stage_bytes(cand) > kStageLimit) break;
    if (total_bytes(cand, 2) > kSmemBudget) break;
    if ((cand - 1) * p->wbox2 + p->tw2 + 128 >= 4096) break;
    const long long tiles = strips * dc_div_up(ho, cand);
    const long long per_max = (tiles + n_sm - 1) / n_sm;
    const int mb = dc_div_up((cand - 1) * p->wbox2 + p->tw2, 128);
    double cost = (double)per_max * (mb + 0.2 + 0.03 * rbox) + 0.15 * rbox;
    if (per_max < 3 && tiles >= 3ll * n_sm) cost *= 1.5;       // too few tiles to overlap the roles
    if (th == 0 || cost < best) { th = cand; best = cost; }
  }
  if (th == 0) return false;
  p->th = th;
  p->rbox = S == 1 ? patch_rows(th) : (patch_rows(th) + 1) / 2;     // rows of one TMA box
  p->tiles_y = dc_div_up(ho, th);
  const long long total_tiles = strips * p->tiles_y;
  const int grid = total_tiles < n_sm ? (int)total_tiles : n_sm;
  p->grid = grid;
  p->tiles_per = (int)(total_tiles / grid);
  p->tiles_rem = (int)(total_tiles % grid);
  p->mb = dc_div_up((th - 1) * p->wbox2 + p->tw2, 128);
  const int th_last = ho - (p->tiles_y - 1) * th;
  p->mb_last = dc_div_up((th_last - 1) * p->wbox2 + p->tw2, 128);
  p->a_stage_bytes = (int)stage_bytes(th);
  p->a_plane_bytes = (int)plane_bytes(th);
  p->a_box_bytes = p->rbox * p->wbox2 * 128;
  const long long per_cta = p->tiles_per + (p->tiles_rem ? 1 : 0);
  int stages = kMaxStages < per_cta ? kMaxStages : (int)per_cta;
  if (stages < 2) stages = 2;
  while (stages > 2 && total_bytes(th, stages) > kSmemBudget) --stages;
  if (total_bytes(th, stages) > kSmemBudget) return false;
  p->stages = stages;
  p->off_out = p->off_a + stages * p->a_stage_bytes;
  p->smem_bytes = (int)total_bytes(th, stages);
  // one instruction per (tap row r, pair shift t, 32-byte K step): where its operand starts in a stage
  int j = 0;
  for (int r = 0; r < g->k; ++r)
    for (int t = 0; t < nt; ++t)
      for (int sl = 0; sl < ko.cch; ++sl, ++j) {
        const uint32_t off = S == 1 ? (uint32_t)((r * p->wbox2 + t) * 128 + sl * 32)
                                    : (uint32_t)((r & 1) * p->a_plane_bytes + ((r >> 1) * p->wbox2 + t) * 128 + sl * 32);
        p->a_lo[j] = (off >> 4) | (1u << 16);    // leading-dimension field: 1 (unused for swizzled K-major)
      }
  return true;
}

}  // namespace

bool dc_conv_pairrows_supported(int n, int h, int w, const dc_geom *g) {
  PairParams p;
  return pair_plan(n, h, w, g, dc_sm_count(), &p);
}

dc_status dc_launch_conv_pairrows(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                                  const float *bias, dc_act act, const void *residual, void *y, void *workspace,
                                  cudaStream_t stream) {
  PairParams p;
  const int n_sm = dc_sm_count();
  if (!pair_plan(n, h, w, g, n_sm, &p)) return DC_ERR_UNSUPPORTED;
  p.act = (int)act;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return DC_ERR_CUDA;
  CUtensorMap map_a;
  {
    // activations: an image row is w/2 lines of 2*c_in channels; the box is 64 channels (128 bytes) wide
    const cuuint64_t C = (cuuint64_t)g->c_in;
    cuuint64_t gdim[4] = {2 * C, (cuuint64_t)(w / 2), (cuuint64_t)h, (cuuint64_t)n};
    cuuint64_t gstr[3] = {4 * C, (cuuint64_t)w * C * 2, (cuuint64_t)h * w * C * 2};
    // stride 2: the box spans 2 * rbox rows and takes every second one
    cuuint32_t box[4] = {64, (cuuint32_t)p.wbox2, (cuuint32_t)(p.stride * p.rbox), 1};
    cuuint32_t es[4] = {1, 1, (cuuint32_t)p.stride, 1};
    CUresult r = encode(&map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(x), gdim, gstr, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return DC_ERR_CUDA;
  }
  static unsigned char attr_done[kDcMaxDevices];
  DC_CUDA_OK(dc_set_max_smem_once(k_conv_tc_pairrows, kSmemBudget, attr_done));
  cudaError_t le = dc_launch_pdl(k_conv_tc_pairrows, dim3(p.grid), dim3(kThreads), (size_t)p.smem_bytes, stream, map_a, p,
                                 w_packed, bias, (const __nv_bfloat16 *)residual, (__nv_bfloat16 *)y,
                                 (DcWsHeader *)workspace);
  if (le != cudaSuccess) return DC_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}
