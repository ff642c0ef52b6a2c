// Weight-streaming GEMM on the 5th-generation tensor cores (tcgen05, accumulators in TMEM,
// operands staged by TMA) for bf16 weights:  out[t, n] = sum_k X[t, k] * W[n, k].
//
// The weight matrix is the MMA "A" operand (128 output features per tile = MMA M), the few
// activation rows are the "B" operand (MMA N = rows padded to a multiple of 16), so a stair
// batch of 1..36 rows costs one pass over the weights.  Both operands are K-major in shared
// memory with the 128-byte swizzle; one pipeline stage holds a 128 x 64 weight tile (16 KB)
// and a Tpad x 64 activation tile.
//
// Work split: the (tile, k-block) space is cut into one contiguous range per CTA (grid = SM
// count), so every SM streams the same number of bytes whatever N and K are.  A tile whose
// k-blocks fall into several CTAs is finished by whichever CTA arrives last: every CTA stores
// its partial tile in a scratch slot, bumps the tile's counter, and the last one adds the
// partials in k order - a fixed order, so results do not depend on arrival order, nor on the
// number of rows in the call.
//
// Warp roles (192 threads): warp 0 issues TMA loads, warp 1 owns TMEM and issues the MMAs,
// warps 2-5 run the epilogue (one TMEM lane quadrant each).  Two accumulator buffers let the
// epilogue of one tile overlap the main loop of the next.  Every wait is bounded by a clock
// limit; on expiry the CTA records STAIRS_ETIMEOUT in the status word, drains its copies,
// frees its TMEM and returns.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "gemm_simt.cuh"

namespace stairs {
namespace tc {

constexpr int BM = 128;          // features per tile
constexpr int BK = 64;           // k elements per stage (one 128-byte swizzle row of bf16)
constexpr int UMMA_K = 16;
constexpr int THREADS = 192;
constexpr int A_STAGE_BYTES = BM * BK * 2;
constexpr int MAX_STAGES = 12;
constexpr int XCH_BYTES = 64 * 16 * 4;   // SwiGLU gate/up exchange, one 16-column chunk
constexpr int SMEM_LIMIT = 232448;       // 227 KB per CTA

enum Epi { TC_STORE_F32 = 0, TC_ADD_F32 = 1, TC_GELU = 2, TC_SWIGLU = 3, TC_LMHEAD = 4 };

struct GemmJob {
  CUtensorMap w_map[3];   // weight sources; box 64 x 128 (k x rows), or 64 x 64 in dual mode
  CUtensorMap x_map;      // activations [rows, K]; box 64 x t_box
  int src_tiles[3];       // tiles per source (dual: tiles of 64 gate + 64 up features)
  int src_col[3];         // first output column of each source
  int n_src;
  int dual;               // 1: rows 0-63 of a tile come from w_map[0], rows 64-127 from w_map[1]
  int n_tiles, t_tiles, kblocks;
  int N;                  // output features (dual: features of one matrix)
  int T;                  // valid activation rows
  int t_box;              // activation rows per tile (MMA N), multiple of 16, <= 256
  int stages;
  int epi;
  float* out_f32; int ldo;      // TC_STORE_F32 / TC_ADD_F32 / TC_LMHEAD (logits, may be null)
  bf16* out_act;                // TC_GELU / TC_SWIGLU, leading dimension ldo
  unsigned long long* keys;     // TC_LMHEAD: packed argmax keys per row
  float* partial;               // [grid][2][t_box][128] scratch for split tiles
  int* counters;                // [n_tiles * t_tiles], zero between calls
  unsigned int* status;         // device status words
  unsigned long long wait_limit;
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false when the clock limit expired or another role raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if ((unsigned long long)(clock64() - t0) > limit) { *abort_flag = 1; return false; }
  }
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar)), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}

__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate, M = 128.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives on the mbarrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor: K-major tile, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffff) >> 4);        // start address, 16-byte units
  d |= (uint64_t)1 << 16;                        // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                        // descriptor version for sm_100
  d |= (uint64_t)2 << 61;                        // SWIZZLE_128B
  return d;
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// k-block range of CTA c out of g over `total` k-blocks
__device__ __forceinline__ long long range_begin(long long total, int c, int g) { return total * c / g; }

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(THREADS, 1) k_gemm_tc(const __grid_constant__ GemmJob job) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int stages = job.stages;
  const int b_stage_bytes = job.t_box * BK * 2;
  const int stage_bytes = A_STAGE_BYTES + b_stage_bytes;
  uint8_t* tail = smem + (size_t)stages * stage_bytes;
  float* xch = reinterpret_cast<float*>(tail);                       // [64][16]
  uint64_t* full = reinterpret_cast<uint64_t*>(tail + XCH_BYTES);    // [stages]
  uint64_t* empty = full + MAX_STAGES;
  uint64_t* acc_full = empty + MAX_STAGES;                           // [2]
  uint64_t* acc_empty = acc_full + 2;                                // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* last_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = gridDim.x, cta = blockIdx.x;
  const long long total = (long long)job.n_tiles * job.t_tiles * job.kblocks;
  const long long kb_begin = range_begin(total, cta, G), kb_end = range_begin(total, cta + 1, G);
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < 2 * job.t_box) tmem_cols <<= 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
    mbar_init(acc_full + 0, 1); mbar_init(acc_full + 1, 1);
    mbar_init(acc_empty + 0, 4); mbar_init(acc_empty + 1, 4);
    *abort_flag = 0; *last_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(tmem_slot, tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // producer bookkeeping (thread 0): loads in flight are drained at teardown after an abort
  int issued = 0, p_stage = 0;
  uint32_t p_phase = 0;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && kb_begin < kb_end) {
      const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
      int& stage = p_stage; uint32_t& phase = p_phase;
      for (long long kb = kb_begin; kb < kb_end; ++kb) {
        const int tile = (int)(kb / job.kblocks), kk = (int)(kb % job.kblocks);
        const int n_tile = tile / job.t_tiles, t_tile = tile % job.t_tiles;
        if (!mbar_wait(empty + stage, phase ^ 1, abort_flag, job.wait_limit)) break;
        uint8_t* a_dst = smem + (size_t)stage * stage_bytes;
        uint8_t* b_dst = a_dst + A_STAGE_BYTES;
        mbar_expect_tx(full + stage, (uint32_t)stage_bytes);
        if (job.dual) {
          tma_load_2d(a_dst, &job.w_map[0], kk * BK, n_tile * 64, full + stage, pol_w);
          tma_load_2d(a_dst + A_STAGE_BYTES / 2, &job.w_map[1], kk * BK, n_tile * 64, full + stage, pol_w);
        } else {
          int s = 0, local = n_tile;
          while (s + 1 < job.n_src && local >= job.src_tiles[s]) { local -= job.src_tiles[s]; ++s; }
          tma_load_2d(a_dst, &job.w_map[s], kk * BK, local * BM, full + stage, pol_w);
        }
        tma_load_2d(b_dst, &job.x_map, kk * BK, t_tile * job.t_box, full + stage, pol_x);
        ++issued;
        if (++stage == stages) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && kb_begin < kb_end) {
      const uint32_t idesc = instr_desc_bf16(job.t_box);
      int stage = 0; uint32_t phase = 0;
      int buf = 0; uint32_t acc_phase[2] = {0, 0};
      bool ok = true;
      for (long long kb = kb_begin; kb < kb_end && ok; ++kb) {
        const int kk = (int)(kb % job.kblocks);
        const bool seg_first = (kb == kb_begin) || kk == 0;
        const bool seg_last = (kb + 1 == kb_end) || kk == job.kblocks - 1;
        if (seg_first) {
          ok = mbar_wait(acc_empty + buf, acc_phase[buf] ^ 1, abort_flag, job.wait_limit);
          if (!ok) break;
          tc_fence_after();
        }
        ok = mbar_wait(full + stage, phase, abort_flag, job.wait_limit);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + (size_t)stage * stage_bytes);
        const uint64_t a_desc = smem_desc_sw128(a_addr), b_desc = smem_desc_sw128(a_addr + A_STAGE_BYTES);
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * job.t_box);
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k)
          umma_bf16(d_tmem, a_desc + (uint64_t)(k * UMMA_K * 2 / 16), b_desc + (uint64_t)(k * UMMA_K * 2 / 16), idesc,
                    (seg_first && k == 0) ? 0u : 1u);
        umma_commit(empty + stage);
        if (seg_last) { umma_commit(acc_full + buf); acc_phase[buf] ^= 1; buf ^= 1; }
        if (++stage == stages) { stage = 0; phase ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;              // TMEM lanes 32*quad .. 32*quad+31
    const int m = quad * 32 + lane;         // row of the tile = feature within the tile
    const int et = threadIdx.x - 64;        // 0..127 within the epilogue group
    int buf = 0; uint32_t acc_phase[2] = {0, 0};
    bool ok = true;
    long long kb = kb_begin;
    while (kb < kb_end && ok) {
      const int tile = (int)(kb / job.kblocks), kk0 = (int)(kb % job.kblocks);
      const int n_tile = tile / job.t_tiles, t_tile = tile % job.t_tiles;
      const long long tile_first = (long long)tile * job.kblocks, tile_end = tile_first + job.kblocks;
      const long long seg_end = tile_end < kb_end ? tile_end : kb_end;
      const bool whole = (kk0 == 0) && (seg_end == tile_end);
      mbar_wait(acc_full + buf, acc_phase[buf], abort_flag, job.wait_limit);
      // one verdict for all 128 epilogue threads: a divergent exit would strand the others at
      // the named barriers below
      epi_bar_sync();
      if (et == 0) *last_flag = *abort_flag ? 0 : 1;
      epi_bar_sync();
      ok = *last_flag != 0;
      epi_bar_sync();
      if (!ok) break;
      acc_phase[buf] ^= 1;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * job.t_box);

      // output column(s) of this thread's feature
      int n_out, n_valid;
      if (job.dual) { n_out = n_tile * 64 + (m & 63); n_valid = n_out < job.N; }
      else {
        int s = 0, local = n_tile;
        while (s + 1 < job.n_src && local >= job.src_tiles[s]) { local -= job.src_tiles[s]; ++s; }
        const int in_src = local * BM + m;
        const int src_n = (s + 1 < job.n_src ? job.src_col[s + 1] : job.N) - job.src_col[s];
        n_out = job.src_col[s] + in_src; n_valid = in_src < src_n;
      }
      const int t_base = t_tile * job.t_box;

      // final epilogue of one 16-column chunk held in v[]
      auto finish = [&](int c0, float* v) {
        if (job.epi == TC_SWIGLU) {
          if (m >= 64) {
#pragma unroll
            for (int j = 0; j < 16; ++j) xch[(m - 64) * 16 + j] = v[j];
          }
          epi_bar_sync();
          if (m < 64 && n_valid) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int t = t_base + c0 + j;
              if (t < job.T) job.out_act[(size_t)t * job.ldo + n_out] = __float2bfloat16_rn(silu_f(v[j]) * xch[m * 16 + j]);
            }
          }
          epi_bar_sync();
          return;
        }
        if (job.epi == TC_LMHEAD) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int t = t_base + c0 + j;   // warp-uniform
            if (t >= job.T) break;
            if (job.out_f32 && n_valid) job.out_f32[(size_t)t * job.ldo + n_out] = v[j];
            unsigned long long key = n_valid ? argmax_key(v[j], (uint32_t)n_out) : 0ull;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
              key = other > key ? other : key;
            }
            if (lane == 0 && key) atomicMax(job.keys + t, key);
          }
          return;
        }
        if (!n_valid) return;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int t = t_base + c0 + j;
          if (t >= job.T) break;
          const size_t o = (size_t)t * job.ldo + n_out;
          if (job.epi == TC_STORE_F32) job.out_f32[o] = v[j];
          else if (job.epi == TC_ADD_F32) job.out_f32[o] += v[j];
          else job.out_act[o] = __float2bfloat16_rn(gelu_erf(v[j]));
        }
      };

      if (whole) {
        for (int c0 = 0; c0 < job.t_box; c0 += 16) {
          float v[16];
          tmem_ld16(taddr + (uint32_t)c0, v);
          finish(c0, v);
        }
        tc_fence_before();
        if (lane == 0) mbar_arrive(acc_empty + buf);
      } else {
        // partial tile: park it, then the last arriver of the tile adds the parts in k order
        const int slot = 2 * cta + (kb == kb_begin ? 0 : 1);
        float* mine = job.partial + (size_t)slot * job.t_box * BM;
        for (int c0 = 0; c0 < job.t_box; c0 += 16) {
          float v[16];
          tmem_ld16(taddr + (uint32_t)c0, v);
#pragma unroll
          for (int j = 0; j < 16; ++j) mine[(size_t)(c0 + j) * BM + m] = v[j];
        }
        tc_fence_before();
        if (lane == 0) mbar_arrive(acc_empty + buf);
        __threadfence();
        epi_bar_sync();
        // CTAs whose ranges touch this tile: first_c .. last_c
        int first_c = (int)((tile_first * G) / total);
        while (range_begin(total, first_c + 1, G) <= tile_first) ++first_c;
        while (first_c > 0 && range_begin(total, first_c, G) > tile_first) --first_c;
        int last_c = first_c;
        while (last_c + 1 < G && range_begin(total, last_c + 1, G) < tile_end) ++last_c;
        const int nseg = last_c - first_c + 1;
        if (et == 0) {
          const int old = atomicAdd(job.counters + tile, 1);
          *last_flag = (old == nseg - 1) ? 1 : 0;
          if (old == nseg - 1) job.counters[tile] = 0;
        }
        epi_bar_sync();
        const bool last = *last_flag != 0;
        epi_bar_sync();
        if (last) {
          __threadfence();
          for (int c0 = 0; c0 < job.t_box; c0 += 16) {
            float v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = 0.f;
            for (int c = first_c; c <= last_c; ++c) {
              const long long cb = range_begin(total, c, G);
              const int sl = 2 * c + (cb >= tile_first ? 0 : 1);
              const float* part = job.partial + (size_t)sl * job.t_box * BM;
#pragma unroll
              for (int j = 0; j < 16; ++j) v[j] += __ldcg(part + (size_t)(c0 + j) * BM + m);
            }
            finish(c0, v);
          }
        }
      }
      buf ^= 1;
      kb = seg_end;
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) {
      *reinterpret_cast<volatile unsigned int*>(job.status + STATUS_ERROR) = 5u;  // STAIRS_ETIMEOUT
      __threadfence_system();
      // loads already issued must land before the shared memory is given back: walk back over
      // the most recent load of every stage and wait (bounded) for its barrier phase
      const long long t0 = clock64();
      int s = p_stage; uint32_t ph = p_phase;
      for (int i = 0; i < stages && i < issued; ++i) {
        if (--s < 0) { s = stages - 1; ph ^= 1; }
        while (!mbar_try(full + s, ph)) {
          if ((unsigned long long)(clock64() - t0) > job.wait_limit) break;
        }
      }
    }
    __syncthreads();
  }
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, tmem_cols); }
}

inline size_t smem_bytes(int t_box, int stages) {
  return 1024 + (size_t)stages * (A_STAGE_BYTES + (size_t)t_box * BK * 2) + XCH_BYTES + (2 * MAX_STAGES + 4) * 8 + 64;
}
inline int pick_stages(int t_box) {
  int s = MAX_STAGES;
  while (s > 2 && smem_bytes(t_box, s) > SMEM_LIMIT) --s;
  return s;
}

}  // namespace tc
}  // namespace stairs
