// One persistent kernel for a whole forward pass over T <= 64 rows (a stairs validation call, an
// assistant step, plain greedy decoding): stair rows, embedding, every layer, LM head, argmax,
// accept - one cooperative launch, one CTA per SM, grid-wide barriers between dependent phases.
//
// Why: at these row counts a layer streams its weights in a few microseconds, so per-kernel
// launch gaps and pipeline fill/drain would dominate.  Here the TMA producer warp of every CTA
// walks a static schedule of weight tiles for the WHOLE pass and keeps the shared-memory ring
// full across phase boundaries: weight tiles (which depend on nothing) are fetched as soon as a
// slot frees up, while the small activation tile of a stage is fetched only once the grid
// barrier that publishes it has completed.  HBM therefore keeps streaming through barriers,
// norms and attention.
//
// Roles per CTA (224 threads): warp 0 = TMA producer, warp 1 = MMA issuer / TMEM owner (GEMM phases, and
// the attention phases' contractions on the tcgen05 path), warps 2-5 = "compute group": GEMM epilogues
// and every non-GEMM phase (rows+embedding, attention softmax and state merge, accept), warp 6 = K/V loader of
// the attention phases.  A GEMM pipeline stage holds one or two 64-element k-blocks, fetched by ONE
// 3-D bulk tensor copy per operand and freed by ONE commit (issue costs, not bandwidth, bound the
// single-thread roles).  GEMM work is cut into contiguous ranges per CTA, in units of two k-blocks
// whatever the stage depth, so results do not depend on the call's row count; a tile cut over
// several CTAs is finished by the CTA that owns its first k-block, which adds the other CTAs' parked
// partial tiles in k order; no flags: a parked word reads as an "empty" pattern until it has been
// stored, and the finisher polls the words it needs.  Normalisation is folded into the GEMMs (operand
// x * gain, epilogue rescales by the row's 1/std from per-tile statistics).
//
// Attention (staircase mask over the paged cache): a unit is (request, kv head, range of 64-position
// chunks, block of queries); all rows x grouped heads of the request share the K/V chunk.  Queries
// (rotated, scaled by log2(e)/sqrt(hd), fp16) and the new positions' K/V are filed by the QKV
// projection's epilogue.  Three ways through a unit, chosen by the host per model and call:
//  - head sizes 64/128, long contexts or many query rows: chunks streamed by the loader warp with
//    tiled bulk copies (128-byte swizzle) through a ring of buffers; S = Q.K^T and O += P.V as
//    tcgen05 MMAs (M = 128 queries, accumulators in TMEM) issued by the MMA warp one chunk ahead of
//    the compute group's base-2 online softmax;
//  - head sizes 64/128 otherwise: the same ring, contractions on fp16 mma.sync tiles, one warp per
//    16-query block, softmax state in registers;
//  - other head sizes: padded tiles staged by 16-byte asynchronous copies from the compute warps.
// Unit boundaries depend only on the request's own committed length, never on the other requests.
//
// With 227 KB of shared memory the L1 is nearly gone: every global or local access is an L2 round
// trip.  Phase descriptors and request geometry are therefore kept in shared memory, cursors in
// scalar registers, and loads that feed a dependent chain are issued together.
//
// All waits (mbarriers, grid barrier, polls of parked sums and states) are clock-bounded: on expiry the CTA
// raises an abort flag (shared memory) and a global abort word that every other CTA's waits poll,
// so the whole grid drains, frees TMEM and exits with STAIRS_ETIMEOUT in the status word.
#pragma once
#include "gemm_tc.cuh"
#include "kernels_basic.cuh"

// Device-side timestamps for tuning (per-phase stamps written to a scratch area while profiling
// is on) are compiled in only with -DSTAIRS_TRACE; the shipped kernel carries none of them.
#ifdef STAIRS_TRACE
#define MK_TRACE_PTR(expr) (expr)
#else
#define MK_TRACE_PTR(expr) (static_cast<unsigned long long*>(nullptr))
#endif

namespace stairs {
namespace mk {

using namespace tc;

enum PhaseKind { PH_EMBED = 0, PH_GEMM = 2, PH_ATTN = 3, PH_PREP = 5, PH_ACCEPT = 6 };

struct Phase {
  int kind, layer;
  // PH_GEMM
  int w_map[3], x_map;
  int src_tiles[3], src_col[3];
  int n_src, dual, n_tiles, kblocks, N, epi, ldo;   // kblocks counts pipeline stages per tile (groups of Params::kps k-blocks)
  int upt;                   // range units (RANGE_UNIT_KB k-blocks) per tile
  void* out;                 // fp32 or bf16 output
  // Normalisation folded into the GEMMs.  norm_in: the activation operand is bf16(x * gain) and
  // the epilogue applies y = rstd_t * (acc - mean_t * u[n]) + c[n] with u = W.gain, c = W.bias
  // (LayerNorm; both NULL for RMSNorm, where y = rstd_t * acc).  next_g: this residual GEMM's
  // finisher also writes bf16(x * next_g) for the following GEMM and per-tile row statistics.
  int ge_max;                // CTAs this GEMM is cut over (0 = all): few tiles are not worth a wide split
  int norm_in;
  int qkv_prep;              // QKV projection: the epilogue rotates, converts and files q, k, v (see epilogue)
  const float* u; const float* c;
  const float* next_g;
  // PH_EMBED
  const float* g;
  // PH_ATTN
  void* kc; void* vc;
};

enum CallMode { CALL_VALIDATE = 0, CALL_DRAFT_FIRST = 1, CALL_DRAFT_NEXT = 2, CALL_PREFILL = 3 };

struct Params {
  const Phase* phases; int n_phases;
  const CUtensorMap* maps;
  int T, t_box, stages;
  int kps;                   // k-blocks (64 k-elements each) per pipeline stage: one TMA box and one commit cover all of them
  int logit_first_row, n_logit_rows;
  // model
  int d, Hq, Hkv, hd, F, vocab, norm_kind, rope; float rope_theta, eps;
  const bf16* tok_emb; const bf16* pos_emb;
  // call
  int mode; int n_req; int slot; int draft_step;
  int draft_first_rows;      // rows of the assistant's first step: 2 (it re-reads the last two committed tokens), or 1 when it shares the main model's cache
  int val_req[64]; int val_k[64]; int val_off[64];   // validate: slot, draft length and first row of each request (a call has <= 64 rows)
  const int* draft; int k_max;
  int* seq; int* n_seq; int max_seq_len;
  int* tok; int* pos; int* req;
  const int* page_table; int page_tokens, max_pages;
  float* x; bf16* h; float* qkv; bf16* o; bf16* ff;
  int lo_row;               // GEMM operands are stored as bf16 hi + bf16 lo; the lo part sits lo_row rows further down
  unsigned long long* keys; int n_keys;
  float4* stats;            // [64 rows][stat_tiles] (mean, M2, count, -) per 128-column tile of x
  int stat_tiles;
  const float* rope_inv;
  int att_dbl;               // attention, copy path: two K/V chunk buffers, the next chunk's copies fly under the current chunk's MMAs
  int att_tma;               // attention, TMA path (head sizes 64 and 128): a loader warp streams K/V chunks through att_nbuf buffers
  int att_nbuf;
  int kv_box_rows;           // rows of one K/V box: min(page_tokens, chunk)
  int att_tc;                // attention on tcgen05 (with att_tma): S = Q.K^T and O += P.V as M = 128 MMAs, accumulators in TMEM
  int att_qblk;              // queries per attention unit: 48 (mma.sync path), 128 (tcgen05 path)
  int att_q_rows;            // tcgen05 path: rows of the Q and P tiles kept in shared memory (queries of a unit, rounded up to 8)
  __half* q16;               // [row][Hq*hd] queries, rotated and scaled by 1/sqrt(hd), written by the QKV epilogue
  float* rope_cs; float* rope_sn;   // [row][hd/2] cos and sin of the call's row positions, written by the embedding phase
     // [hd/2] theta^(-2i/hd)
  float* logits;            // optional dump
  int* target_tokens; int* accept_len; int commit; int* draft_out;
  // scratch
  float* partial; int* counters;
  float* attn_part;         // two sets of [units][QBLK][hd + 4]: O, running max, running sum, pad; every word PARTIAL_EMPTY between uses
  int attn_part_units;
  size_t attn_set_stride;   // floats between the two sets of parked states (alternate attention phases)
  unsigned long long* bar;  // [0] arrivals (monotonic), [1] abort word
  unsigned long long bar_base;
  unsigned int* status; unsigned long long wait_limit;
  unsigned long long* trace;   // optional: per phase {start, work done, arrived} ns timestamps of CTA 0 and of the last CTA
};

constexpr int MK_THREADS = THREADS + 32;   // the GEMM kernel's six warps plus the K/V loader of the attention phases
constexpr int MAX_KV_BUF = 4;
constexpr int ATT_CHUNK = 64;
constexpr int ATT_QBLK = 48;                    // queries per unit on the mma.sync path
constexpr int ATT_QBLK_TC = 128;                // ... on the tcgen05 path (the MMA's M)
constexpr int VT_LD = 132;                      // row pitch (floats) of the epilogue's 16 x 128 exchange tile
constexpr int MK_XCH_BYTES = 16 * VT_LD * 4;     // the tile itself

struct AttnSmem {   // carved after the GEMM ring: Q block (bf16), K and V chunk tiles (bf16), merge buffer (fp32)
  static __host__ __device__ size_t k_pitch(int hd) { return (size_t)hd * 2 + 16; }
  static __host__ __device__ size_t q_bytes(int hd) { return (size_t)ATT_QBLK * k_pitch(hd); }
  static __host__ __device__ size_t kv_bytes(int hd) { return (size_t)ATT_CHUNK * k_pitch(hd); }
  static __host__ __device__ size_t merge_bytes(int hd) { return (size_t)16 * (hd + 4) * 4 + 64; }
  // TMA path: a chunk buffer holds K then V, each as hd / 64 column halves of [CHUNK rows][128 bytes] with the 128-byte swizzle
  static __host__ __device__ size_t kv_buf_bytes(int hd) { return (size_t)2 * ATT_CHUNK * hd * 2; }
  // copy path: Q block, then one or two padded K/V buffers; TMA path: nbuf chunk buffers (1024-byte aligned), then the Q block
  // tcgen05 path (tc_q_rows > 0): Q tile (hd / 64 halves of [q_rows][128 bytes]) and P tile ([q_rows][128 bytes]),
  // both swizzled, then the chunk buffers; an M = 128 MMA reads 128 rows from a tile's start, so at
  // least 16 KB of this region must follow the P tile: the first chunk buffer does
  static __host__ __device__ size_t tc_head_bytes(int hd, int q_rows) { return (size_t)(hd / 64 + 2) * q_rows * 128; }   // Q halves, two P tiles
  static __host__ __device__ size_t bytes(int hd, int dbl, int tma, int nbuf, int tc_q_rows = 0) {
    if (tc_q_rows > 0) return 1024 + tc_head_bytes(hd, tc_q_rows) + (size_t)nbuf * kv_buf_bytes(hd) + 64;
    return tma ? 1024 + (size_t)nbuf * kv_buf_bytes(hd) + q_bytes(hd) + 64 : q_bytes(hd) + (dbl ? 4 : 2) * kv_bytes(hd) + 64;
  }
};

// 16-byte asynchronous copy global -> shared; `on` false writes zeros and reads nothing
__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool on) {
  const uint32_t n = on ? 16u : 0u;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

// mma.sync m16n8k16 (fp16 in, fp32 accumulate) and its operand loads, for the attention tiles:
// queries, cached K/V and the softmax weights are fp16 (11 significant bits)
__device__ __forceinline__ void mma_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t* r, const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(p)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t* r, const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(p)));
}
// 2^x by the hardware approximation (relative error about 2^-22; the softmax weights are rounded
// to fp16 afterwards).  Scores are kept in the base-2 domain: the queries carry log2(e) / sqrt(hd).
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// Split-tile partial sums travel without a flag: a slot element holds PARTIAL_EMPTY (a NaN pattern that
// arithmetic never produces - the hardware's NaN is 0x7fffffff) until its producer stores the sum, the
// consumer polls the elements it needs and puts the pattern back.  Element-wise relaxed accesses at GPU scope.
constexpr uint32_t PARTIAL_EMPTY = 0xffffffffu;
__device__ __forceinline__ void st_relaxed_f32(float* p, float v) {
  asm volatile("st.relaxed.gpu.global.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}
__device__ __forceinline__ uint4 ld_relaxed_u4(const float* p) {
  uint4 v;
  asm volatile("ld.relaxed.gpu.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint2 ld_relaxed_u2(const float* p) {
  uint2 v;
  asm volatile("ld.relaxed.gpu.global.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed_u4(float* p, uint4 v) {
  asm volatile("st.relaxed.gpu.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void red_release_add_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.global;" ::: "memory"); }   // (global memory is all these fences are about)
// the same for this CTA's shared memory only (tiles written with plain stores, read by the tensor core)
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}

// Range of pipeline stages of this CTA in a GEMM phase.  The (tile, k) space is cut in UNITS of
// RANGE_UNIT_KB k-blocks whatever the stage depth of the launch is, so that a tile's segment
// boundaries - and with them the order of the fp32 additions - do not depend on the row count of
// the call (calls with more rows use shallower stages): a request gives bit-identical results
// alone and inside a larger batch.  The phase is cut over min(G, units) CTAs so that no
// participating range is empty (the split-tile bookkeeping counts one segment per CTA touching a tile).
constexpr int RANGE_UNIT_KB = 2;
struct KRange { int begin, end; int ge; };   // 32-bit throughout: units * CTAs < 2^32 is checked on the host, and 64-bit divisions are long code
// first stage of unit u: upt units and spt stages per tile, spu stages per unit (the last unit of a tile may be short)
__device__ __forceinline__ int unit_to_stage(unsigned u, int upt, int spt, int spu) {
  if (spu == 1) return (int)u;
  const unsigned tile = u / (unsigned)upt;
  const int j = (int)(u - tile * (unsigned)upt);
  return (int)tile * spt + (j * spu < spt ? j * spu : spt);
}
__device__ __forceinline__ KRange phase_range(int n_tiles, int upt, int spt, int spu, int cta, int G, int ge_max) {
  KRange r;
  const unsigned total = (unsigned)n_tiles * (unsigned)upt;
  if (ge_max > 0 && ge_max < G) G = ge_max;
  r.ge = (int)(total < (unsigned)G ? total : (unsigned)G);
  if (cta >= r.ge) { r.begin = r.end = 0; return r; }
  r.begin = unit_to_stage((total * (unsigned)cta) / (unsigned)r.ge, upt, spt, spu);
  r.end = unit_to_stage((total * (unsigned)(cta + 1)) / (unsigned)r.ge, upt, spt, spu);
  return r;
}

// GEMM activation operands keep ~16 mantissa bits: value = hi + lo with hi = bf16(value) and
// lo = bf16(value - hi); the MMAs run once on each part into the same accumulator.
__device__ __forceinline__ void store_split(bf16* base, size_t idx, size_t lo_off, float v) {
  const bf16 hi = __float2bfloat16_rn(v);
  base[idx] = hi;
  base[idx + lo_off] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// Four consecutive values as bf16 hi parts and bf16 lo parts (8-byte stores; idx a multiple of 4).
__device__ __forceinline__ void store_split4(bf16* base, size_t idx, size_t lo_off, float4 v) {
  const __nv_bfloat162 h01 = __floats2bfloat162_rn(v.x, v.y), h23 = __floats2bfloat162_rn(v.z, v.w);
  *reinterpret_cast<uint2*>(base + idx) = make_uint2(*reinterpret_cast<const uint32_t*>(&h01), *reinterpret_cast<const uint32_t*>(&h23));
  *reinterpret_cast<uint2*>(base + idx + lo_off) =
      make_uint2(pack_bf16x2(v.x - __low2float(h01), v.y - __high2float(h01)), pack_bf16x2(v.z - __low2float(h23), v.w - __high2float(h23)));
}

// Sums 32 per-lane values across the warp, all at once: on return lane l holds the warp-wide
// total of a[l].  Each halving step exchanges the half a lane does not keep (31 shuffles in five
// dependent steps, instead of 32 separate five-step reductions).
__device__ __forceinline__ float warp_multi_sum32(float (&a)[32], int lane) {
#pragma unroll
  for (int h = 16; h >= 1; h >>= 1) {
    const bool up = (lane & h) != 0;
#pragma unroll
    for (int i = 0; i < h; ++i) {
      const float send = up ? a[i] : a[i + h];
      const float keep = up ? a[i + h] : a[i];
      a[i] = keep + __shfl_xor_sync(0xffffffffu, send, h);
    }
  }
  return a[0];
}

// Geometry of one request's attention units.
struct AttnReq { int slot, base, R, off, n_chunks, cpu, n_ranges, n_qblk, units; };

// Shared per-CTA control block.
struct Ctl {
  uint64_t full[MAX_STAGES], empty[MAX_STAGES], acc_full[2], acc_empty[2];
  uint64_t kv_full[MAX_KV_BUF], kv_empty[MAX_KV_BUF];   // attention K/V chunk buffers (TMA path)
  // tcgen05 attention: S of a chunk is in TMEM (two S buffers) / the chunk's P tile is written and O rescaled
  // (two P tiles; one arrival per compute warp) / the unit's Q tile is staged / a P.V has completed
  uint64_t s_full[2], p_full[2], q_full, o_done;
  volatile int areq_ready;                              // the requests' attention geometry below is filled in
  uint32_t tmem_slot;
  volatile int abort_flag;
  volatile int bcast;
  float rstd[64], mu[64];       // per-row statistics of the current norm_in GEMM phase
  int rowbase[2][64];           // attention staging: cache row of each position of the chunk (per chunk buffer)
  AttnReq areq[64];             // per request, filled once per launch (a request has at least one row: <= 64)
  alignas(16) uint32_t phc[2][(sizeof(Phase) + 3) / 4];   // this and the next phase's descriptor (global memory is a
                                                          // long round trip with the L1 carved down to almost nothing)
  alignas(16) float gtile[128]; // next operand's gain for the current tile's columns
  alignas(16) float utile[128]; // folded-normalisation constants u[n], c[n] of the tile's columns
  alignas(16) float ctile[128];
};

// Uniform verdict for the 128 compute threads after any of them may have timed out in a wait:
// a divergent exit would strand the others at a named barrier.
__device__ __forceinline__ bool group_ok(Ctl* ctl, int et) {
  epi_bar_sync();
  if (et == 0) ctl->bcast = ctl->abort_flag ? 0 : 1;
  epi_bar_sync();
  return ctl->bcast != 0;
}

struct Waiter {
  volatile int* abort_flag; const unsigned long long* gabort; unsigned long long limit;
  unsigned int* status;   // host-visible status words: [1] kind of the first wait that ran out, [2..5] where
  // the first expired wait of a launch leaves a note for the host's error text (plain accesses: the
  // words live in mapped host memory; a lost race only costs detail)
  __device__ __forceinline__ void note(unsigned int kind, unsigned int a, unsigned int b, unsigned int c, unsigned int d) const {
    volatile unsigned int* s = status;
    if (s[STATUS_WHERE] == 0u) { s[STATUS_WHERE] = kind; s[2] = a; s[3] = b; s[4] = c; s[5] = d; }
  }
  __device__ __forceinline__ bool poll_abort(long long t0) const {
    if (*abort_flag) return true;
    if ((unsigned long long)(clock64() - t0) > limit) { *abort_flag = 1; return true; }
    return false;
  }
  // mbarrier wait (bounded).  The polling loops are kept out of line: they are inlined nowhere, so the
  // many wait sites cost a test and a call each instead of a copy of the loop (the kernel's code has
  // to stay inside the instruction cache: every phase runs its code once, and code that misses runs
  // at a fraction of the warm issue rate).
  __device__ __noinline__ bool wait_slow(uint64_t* bar, uint32_t parity) const {
    const long long t0 = clock64();
    int spins = 0;
    while (true) {
      if (mbar_try(bar, parity)) return true;
      if (poll_abort(t0)) {
        if ((unsigned long long)(clock64() - t0) > limit) note(1u, (unsigned)blockIdx.x, (unsigned)threadIdx.x, parity, 0u);
        return false;
      }
      if ((++spins & 255) == 0 && ld_acquire_u64(gabort)) { *abort_flag = 1; return false; }
    }
  }
  __device__ __forceinline__ bool wait(uint64_t* bar, uint32_t parity) const {
    if (mbar_try(bar, parity)) return true;
    return wait_slow(bar, parity);
  }
  // grid barrier wait: arrivals >= target
  __device__ __noinline__ bool wait_grid(const unsigned long long* counter, unsigned long long target) const {
    const long long t0 = clock64();
    int spins = 0;
    while (ld_acquire_u64(counter) < target) {
      if (poll_abort(t0)) {
        if ((unsigned long long)(clock64() - t0) > limit) note(2u, (unsigned)blockIdx.x, (unsigned)threadIdx.x, (unsigned)target, 0u);
        return false;
      }
      if ((++spins & 63) == 0 && ld_acquire_u64(gabort)) { *abort_flag = 1; return false; }
    }
    return true;
  }
};

// Cursor over one CTA's pipeline stages of all GEMM phases, in program order (the TMA producer keeps
// two, one for weight tiles and one for activation tiles).  Per-phase fields
// are hoisted into registers on phase entry; tile and k indices advance incrementally.  Scalar
// fields only: an array indexed at run time would put the cursor in local memory, and with the L1
// carved down for shared memory every such access is an L2 round trip.
struct WCursor {
  int ph, kk, n_tile, remaining, kblocks, dual, n_src, x_map;
  int st0, st1, wmap0, wmap1, wmap2;   // tiles of sources 0 and 1; tensor-map indices of the (up to) three sources
  const CUtensorMap* wm0; int row;
  bool valid;
  __device__ __forceinline__ void locate(const Params& P) {   // source map and row coordinate of tile n_tile
    if (dual) { wm0 = P.maps + wmap0; row = n_tile * BM; }   // gate and up rows interleaved by the host: 64 + 64 per tile
    else {
      int local = n_tile, wm = wmap0;
      if (n_src > 1 && local >= st0) {
        local -= st0; wm = wmap1;
        if (n_src > 2 && local >= st1) { local -= st1; wm = wmap2; }
      }
      wm0 = P.maps + wm; row = local * BM;
    }
  }
  __device__ __forceinline__ void enter(const Params& P, int cta, int G, int from) {   // first GEMM phase >= from in which this CTA has work
    for (int p_i = from; p_i < P.n_phases; ++p_i) {
      const Phase& p = P.phases[p_i];
      if (p.kind != PH_GEMM) continue;
      const KRange kr = phase_range(p.n_tiles, p.upt, p.kblocks, RANGE_UNIT_KB / P.kps, cta, G, p.ge_max);
      if (kr.begin >= kr.end) continue;
      ph = p_i; kblocks = p.kblocks; dual = p.dual; n_src = p.n_src; x_map = p.x_map;
      st0 = p.src_tiles[0]; st1 = p.src_tiles[1];
      wmap0 = p.w_map[0]; wmap1 = p.w_map[1]; wmap2 = p.w_map[2];
      n_tile = kr.begin / p.kblocks; kk = kr.begin - n_tile * p.kblocks;
      remaining = kr.end - kr.begin;
      locate(P);
      valid = true;
      return;
    }
    valid = false;
  }
  __device__ __forceinline__ void advance(const Params& P, int cta, int G) {
    if (--remaining == 0) { enter(P, cta, G, ph + 1); return; }
    if (++kk == kblocks) { kk = 0; ++n_tile; locate(P); }
  }
};

// Asks L2 for one weight tile ahead of the shared-memory ring (no shared memory, no barrier involved).
__device__ __forceinline__ void tma_load_2d_nohint(void* dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar)) : "memory");
}
// Tiled 3-D load global -> shared.  The operand matrices [rows, K] are described to TMA as
// [K / 64][rows][64]: a box of (64, rows of the tile, kps) lands as kps consecutive K-major slabs
// with the 128-byte swizzle, i.e. several k-blocks per copy instruction.
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, uint64_t* bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(bar)), "l"(policy) : "memory");
}

// ---------------------------------------------------------------------------------------------
// Row helpers
// ---------------------------------------------------------------------------------------------
struct RowInfo { int tok, pos, slot; };

__device__ __forceinline__ RowInfo row_info(const Params& P, int t) {
  RowInfo r;
  auto clampv = [&](int v) { return v < 0 ? 0 : (v >= P.vocab ? P.vocab - 1 : v); };
  if (P.mode == CALL_VALIDATE) {
    int i = 0;
    while (i + 1 < P.n_req && P.val_off[i + 1] <= t) ++i;
    const int rr = t - P.val_off[i];
    r.slot = P.val_req[i];
    const int base = P.n_seq[r.slot] - 1;
    r.pos = base + rr;
    r.tok = clampv(rr == 0 ? P.seq[(size_t)r.slot * P.max_seq_len + base] : P.draft[i * P.k_max + rr - 1]);
  } else if (P.mode == CALL_PREFILL) {
    // T consecutive prompt positions starting at draft_step (no logits are taken)
    r.slot = P.slot;
    r.pos = P.draft_step + t;
    r.tok = clampv(P.seq[(size_t)P.slot * P.max_seq_len + r.pos]);
  } else if (P.mode == CALL_DRAFT_FIRST) {
    r.slot = P.slot;
    const int n = P.n_seq[P.slot];
    r.pos = n - P.draft_first_rows + t;
    r.tok = clampv(P.seq[(size_t)P.slot * P.max_seq_len + r.pos]);
  } else {
    r.slot = P.slot;
    r.pos = P.n_seq[P.slot] - 1 + P.draft_step;
    r.tok = clampv(P.draft[P.draft_step - 1]);
  }
  return r;
}

// Row of the K/V pools that holds the position of the call's row t.
__device__ __forceinline__ int cache_row_of(const Params& P, int t) {
  int slot, pos;
  if (P.mode == CALL_VALIDATE) {
    int i = 0;
    while (i + 1 < P.n_req && P.val_off[i + 1] <= t) ++i;
    slot = P.val_req[i]; pos = P.n_seq[slot] - 1 + (t - P.val_off[i]);
  } else if (P.mode == CALL_PREFILL) { slot = P.slot; pos = P.draft_step + t; }
  else if (P.mode == CALL_DRAFT_FIRST) { slot = P.slot; pos = P.n_seq[slot] - P.draft_first_rows + t; }
  else { slot = P.slot; pos = P.n_seq[slot] - 1 + P.draft_step; }
  return P.page_table[(size_t)slot * P.max_pages + pos / P.page_tokens] * P.page_tokens + pos % P.page_tokens;
}

// sum over the 128 compute threads (4 warps); red = 4 floats
__device__ __forceinline__ float group_sum(float v, float* red, int et) {
  v = warp_sum(v);
  epi_bar_sync();
  if ((et & 31) == 0) red[et >> 5] = v;
  epi_bar_sync();
  return red[0] + red[1] + red[2] + red[3];
}

// Row t of the residual stream from the embedding tables, the next GEMM's operand bf16(x * g)
// and the row's statistics (one entry covering the whole row), by the 128 compute threads.
__device__ void embed_row(const Params& P, int t, const RowInfo& r, const float* g, float* red, int et) {
  const int d = P.d;
  float* xr = P.x + (size_t)t * d;
  bf16* hr = P.h + (size_t)t * d;
  const bf16* e = P.tok_emb + (size_t)r.tok * d;
  const bf16* pe = P.pos_emb ? P.pos_emb + (size_t)r.pos * d : nullptr;
  // (rolled loops: this runs once per row and call, and code that is executed once costs its
  // instruction fetch - the second pass re-reads this thread's own stores instead of keeping
  // the row in registers)
  float s1 = 0.f;
#pragma unroll 4
  for (int col = et; col < d; col += 128) {
    float v = __bfloat162float(e[col]);
    if (pe) v += __bfloat162float(pe[col]);
    xr[col] = v;
    store_split(hr, col, (size_t)P.lo_row * d, v * g[col]);
    s1 += v;
  }
  const float mean = group_sum(s1, red, et) / (float)d;
  float s2 = 0.f;
#pragma unroll 4
  for (int col = et; col < d; col += 128) { const float c = xr[col] - mean; s2 += c * c; }
  const float m2 = group_sum(s2, red, et);
  for (int tile = et; tile < P.stat_tiles; tile += 128)
    P.stats[(size_t)t * P.stat_tiles + tile] = tile == 0 ? make_float4(mean, m2, (float)d, 0.f) : make_float4(0.f, 0.f, 0.f, 0.f);
  if (P.rope && et < P.hd / 2) {   // rotation table of this row's position, shared by every layer
    float sn, cs;
    sincosf((float)r.pos * P.rope_inv[et], &sn, &cs);
    P.rope_cs[(size_t)t * (P.hd / 2) + et] = cs;
    P.rope_sn[(size_t)t * (P.hd / 2) + et] = sn;
  }
}

// ---------------------------------------------------------------------------------------------
// Attention units
// ---------------------------------------------------------------------------------------------

__device__ __forceinline__ AttnReq attn_req(const Params& P, int i, int G) {
  AttnReq a;
  if (P.mode == CALL_VALIDATE) {
    a.slot = P.val_req[i]; a.R = P.val_k[i] + 1; a.off = P.val_off[i];
    a.base = P.n_seq[a.slot] - 1;
  } else if (P.mode == CALL_PREFILL) {
    a.slot = P.slot; a.R = P.T; a.off = 0; a.base = P.draft_step;
  } else if (P.mode == CALL_DRAFT_FIRST) {
    a.slot = P.slot; a.R = P.draft_first_rows; a.off = 0; a.base = P.n_seq[P.slot] - P.draft_first_rows;
  } else {
    a.slot = P.slot; a.R = 1; a.off = 0; a.base = P.n_seq[P.slot] - 1 + P.draft_step;
  }
  a.n_chunks = (a.base + a.R + ATT_CHUNK - 1) / ATT_CHUNK;
  // chunks per unit: from the first row's position only (so it is the same for any draft length)
  const int c0 = (a.base + ATT_CHUNK) / ATT_CHUNK;
  int cpu = 1;
  while (cpu < 64 && P.Hkv * ((c0 + cpu - 1) / cpu) > G) cpu <<= 1;   // one unit per CTA where possible: a unit's fixed cost exceeds a chunk's
  a.cpu = cpu;
  a.n_ranges = (a.n_chunks + cpu - 1) / cpu;
  a.n_qblk = (a.R * (P.Hq / P.Hkv) + P.att_qblk - 1) / P.att_qblk;
  a.units = P.Hkv * a.n_ranges * a.n_qblk;
  return a;
}


// Consumer side of the K/V chunk ring of the TMA path: buffer and parity of the next chunk; parity of
// the tcgen05 path's MMA-completion barrier.
struct KvCons { int buf; uint32_t par; uint32_t sc; uint32_t o_par; };   // sc: chunks of the tcgen05 path so far (S / P buffer = sc & 1)

// First chunk buffer of the TMA paths (1024-byte aligned; the tcgen05 path keeps its Q and P tiles in front of it).
__device__ __forceinline__ uint8_t* att_ring_base(const Params& P, uint8_t* att_smem) {
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(att_smem) + 1023) & ~(uintptr_t)1023);
  return P.att_tc ? base + AttnSmem::tc_head_bytes(P.hd, P.att_q_rows) : base;
}

// One attention unit, executed by the 128 compute threads (4 warps), on the legacy tensor path
// (mma.sync m16n8k16).  The unit's queries are cut into blocks of 16 (one MMA M tile), one warp
// per block: S = Q.K^T, online softmax per row with quad shuffles, O += P.V with P reused from
// the accumulator registers and V fetched with ldmatrix.trans; softmax state and output
// accumulators never leave the warp's registers.  With one or two blocks the warps also split
// each chunk's positions in two and merge once per unit.  The block's result is either final
// (the unit saw every visible position) or parked for the merge at the end of the attention phase.
//
// K/V chunks of 64 positions reach shared memory in one of two ways.  TMA path (head sizes 64 and
// 128): the loader warp streams them through a ring of buffers with tiled bulk copies (one box per
// page slice and 64-column half, 128-byte swizzle) and this function only waits on the ring's
// barriers - chunks of already cached positions are in flight before the phase even starts.
// Copy path (other head sizes): the compute threads stage padded tiles with 16-byte asynchronous
// copies, cache rows looked up once per chunk.
template <bool TMA>
__device__ void attn_unit(const Params& P, const Phase& ph, const AttnReq& a, int kvh, int range, int qblk, int part_slot, int part_set,
                          uint8_t* att_smem, Ctl* ctl, int et, bool& ok, KvCons& kvc, const Waiter& W,
                          unsigned long long* tra) {
  const int hd = P.hd, G = P.Hq / P.Hkv, nkv = P.Hkv * hd, nq = P.Hq * hd;
  const int lane = et & 31, w = et >> 5, g = lane >> 2, t4 = lane & 3;
  const int Q = a.R * G;
  const int q0 = qblk * ATT_QBLK, nQ = min(ATT_QBLK, Q - q0);
  const size_t pitch = AttnSmem::k_pitch(hd);               // padded row pitch (queries; K/V of the copy path)
  const size_t kvb = AttnSmem::kv_bytes(hd);
  const size_t kvbuf = AttnSmem::kv_buf_bytes(hd);
  // TMA path: ring of chunk buffers (1024-byte aligned) then the Q block; copy path: Q block then padded buffers
  uint8_t* ring = att_ring_base(P, att_smem);
  uint8_t* qs = TMA ? ring + (size_t)P.att_nbuf * kvbuf : att_smem;   // [QBLK][pitch] fp16, rotated and pre-scaled
  uint8_t* kv0 = qs + AttnSmem::q_bytes(hd);                // copy path, buffer b: K [CHUNK][pitch] then V, at kv0 + b * 2 * kvb
  uint8_t* ks = kv0;                                        // the buffer being computed on
  uint8_t* vs = ks + kvb;
  __half* kc = reinterpret_cast<__half*>(ph.kc);
  __half* vc = reinterpret_cast<__half*>(ph.vc);
  const int* pt = P.page_table + (size_t)a.slot * P.max_pages;
  const int ksteps = hd / 16, ntiles = hd / 8;

  const int c_begin = range * a.cpu, c_end = min(a.n_chunks, c_begin + a.cpu);
  const int n_mt = (nQ + 15) / 16;
  const int pieces = hd * 2 / 16;   // 16-byte pieces per row

  // the unit's queries: query index q -> row r = q / G, head = kvh * G + q % G; rows past the unit's queries are zero
  auto stage_q = [&]() {
    const int dj = 128 / pieces, dp = 128 % pieces;
    int ql = et / pieces, pc = et % pieces;
    while (ql < ATT_QBLK) {
      const bool on = ql < nQ;
      const int q = on ? q0 + ql : q0;
      cp_async16(qs + (size_t)ql * pitch + pc * 16,
                 reinterpret_cast<const uint4*>(P.q16 + (size_t)(a.off + q / G) * nq + (size_t)(kvh * G + q % G) * hd) + pc, on);
      ql += dj; pc += dp;
      if (pc >= pieces) { pc -= pieces; ++ql; }
    }
  };
  // Copy path: stages chunk c (and, with the unit's first chunk, its queries) with 16-byte
  // asynchronous copies issued by all 128 threads (no registers held, so all of a thread's copies
  // are in flight together; rows past the end are zero-filled by the copy itself).  The rows of
  // this call's new positions are in the cache already: the QKV epilogue put them there.
  auto stage_issue = [&](int c, int b, bool with_q) {
    const int p0 = c * ATT_CHUNK;
    const int n_pos = min(ATT_CHUNK, a.base + a.R - p0);
    uint8_t* kd = kv0 + (size_t)b * 2 * kvb;
    uint8_t* vd = kd + kvb;
    int* rowbase = ctl->rowbase[b];
    // cache row of each position of the chunk, looked up once (-1: past the end)
    if (et < ATT_CHUNK) {
      const int pz = p0 + et;
      rowbase[et] = et < n_pos ? pt[pz / P.page_tokens] * P.page_tokens + (pz % P.page_tokens) : -1;
    }
    epi_bar_sync();
    {
      // items (row, 16-byte piece) et, et + 128, ...; row and piece advance without divisions
      const int dj = 128 / pieces, dp = 128 % pieces;
      int jr = et / pieces, pc = et % pieces;
      const size_t head_off = (size_t)kvh * hd;
      while (jr < ATT_CHUNK) {
        const int rb = rowbase[jr];
        const bool on = rb >= 0;
        const size_t off = (size_t)(on ? rb : 0) * nkv + head_off;
        cp_async16(kd + jr * pitch + pc * 16, reinterpret_cast<const uint4*>(kc + off) + pc, on);
        cp_async16(vd + jr * pitch + pc * 16, reinterpret_cast<const uint4*>(vc + off) + pc, on);
        jr += dj; pc += dp;
        if (pc >= pieces) { pc -= pieces; ++jr; }
      }
    }
    if (with_q) stage_q();
    cp_async_commit();
  };

  if (tra) tra[1] = globaltimer_ns();
  if (TMA) { stage_q(); cp_async_commit(); }
  else stage_issue(c_begin, 0, true);
  if (tra) tra[2] = globaltimer_ns();

  // Warp w owns query block (MMA M tile) w of the unit and walks the chunk's four 16-position
  // slices itself, so its softmax state and output accumulators never leave its registers.
  // With one or two query blocks the four warps also split each chunk's positions in two (warps
  // 0, 1 take the first 32 positions, warps 2, 3 the last 32) and the two states of a block are
  // merged once, at the end of the unit.
  const int ps = (n_mt <= 2 && hd >= 64) ? 2 : 1;
  const int mt = ps == 2 ? (w & 1) : w, part = ps == 2 ? (w >> 1) : 0;
  const bool active = mt < n_mt;
  const int ql_a = mt * 16 + g, ql_b = ql_a + 8;
  const int last_a = (active && ql_a < nQ) ? a.base + (q0 + ql_a) / G : -1;   // last visible position
  const int last_b = (active && ql_b < nQ) ? a.base + (q0 + ql_b) / G : -1;
  float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
  float o[16][4];
#pragma unroll
  for (int nd = 0; nd < 16; ++nd) { o[nd][0] = o[nd][1] = o[nd][2] = o[nd][3] = 0.f; }

  int cur = 0;
  int hold_buf = -1;   // TMA path: the last chunk's buffer is kept (it serves the merge) and released at the end
  for (int c = c_begin; c < c_end && ok; ++c) {
    if (TMA) {
      if (c == c_begin) { cp_async_wait_all(); epi_bar_sync(); }   // the queries
      cur = kvc.buf;
      if (!W.wait(ctl->kv_full + cur, kvc.par)) { ok = false; break; }   // (the verdict is made uniform after the loop)
      __syncwarp();
      ks = ring + (size_t)cur * kvbuf; vs = ks + kvbuf / 2;
      if (++kvc.buf == P.att_nbuf) { kvc.buf = 0; kvc.par ^= 1u; }
    } else {
      // with two chunk buffers the next chunk's copies are issued before this chunk is waited for
      const bool ahead = P.att_dbl && c + 1 < c_end;
      if (ahead) { stage_issue(c + 1, cur ^ 1, false); cp_async_wait_but_one(); }
      else cp_async_wait_all();
      epi_bar_sync();
      ks = kv0 + (size_t)cur * 2 * kvb; vs = ks + kvb;
    }
    if (tra && c == c_begin) tra[4] = globaltimer_ns();
    const int p0 = c * ATT_CHUNK;
    const int n_pos = min(ATT_CHUNK, a.base + a.R - p0);
    const bool all_visible = p0 + ATT_CHUNK - 1 <= a.base;   // (then n_pos is a whole chunk too)
    // address of the 16-byte piece `piece` of row j of a K or V tile: padded rows (copy path) or
    // 64-column halves of 128-byte rows with the 128-byte swizzle (TMA path)
    auto kv_addr = [&](const uint8_t* base, int j, int piece) -> const uint8_t* {
      if (TMA) return base + (size_t)(piece >> 3) * (ATT_CHUNK * 128) + (size_t)j * 128 + (size_t)(((piece & 7) ^ (j & 7)) << 4);
      return base + (size_t)j * pitch + (size_t)piece * 16;
    };
    if (active) {
      // 32 positions (two MMA k-steps of P.V, four n-tiles of S) per round: four independent
      // accumulator chains hide the MMA latency, and the softmax bookkeeping is done once per 32
      for (int sl0 = 32 * part; sl0 < n_pos; sl0 += 32 * ps) {
        float sc[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f; }
        // Operand fragments by ldmatrix: for the queries one x4 per k-step (rows 0-7 / 8-15 of
        // the block x the k-step's two 8-column halves), for K one x4 per pair of 8-position
        // n-tiles (positions x the two halves).  Lane l supplies the address of matrix l / 8,
        // row l % 8.
        const uint8_t* q_lane = qs + (size_t)(mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * pitch + (lane >> 4) * 16;
        const int k_row = sl0 + (lane & 7) + (lane >> 4) * 8, k_pc = (lane >> 3) & 1;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          if (kk < ksteps) {
            uint32_t af[4], kf0[4], kf1[4];
            ldmatrix_x4(af, q_lane + kk * 32);
            ldmatrix_x4(kf0, kv_addr(ks, k_row, kk * 2 + k_pc));
            ldmatrix_x4(kf1, kv_addr(ks, k_row + 16, kk * 2 + k_pc));
            mma_16816(sc[0], af, kf0[0], kf0[1]);
            mma_16816(sc[1], af, kf0[2], kf0[3]);
            mma_16816(sc[2], af, kf1[0], kf1[1]);
            mma_16816(sc[3], af, kf1[2], kf1[3]);
          }
        }
        // staircase mask (rows past the chunk's last position hold stale data: assigned, never
        // computed with), row maxima.  A chunk of positions cached before this call is visible to
        // every query as a whole and needs no mask.
        float mx_a = -INFINITY, mx_b = -INFINITY;
        if (all_visible) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            mx_a = fmaxf(mx_a, fmaxf(sc[j][0], sc[j][1])); mx_b = fmaxf(mx_b, fmaxf(sc[j][2], sc[j][3]));
          }
          // (rows past the unit's queries hold zero queries: they run along harmlessly and are never written)
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int jl = sl0 + 8 * j + t4 * 2 + e, pj = p0 + jl;
              const bool in = jl < n_pos;
              if (!(in && pj <= last_a)) sc[j][e] = -INFINITY;
              if (!(in && pj <= last_b)) sc[j][2 + e] = -INFINITY;
              mx_a = fmaxf(mx_a, sc[j][e]); mx_b = fmaxf(mx_b, sc[j][2 + e]);
            }
          }
        }
        mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1)); mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
        mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1)); mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
        const float mn_a = fmaxf(m_a, mx_a), mn_b = fmaxf(m_b, mx_b);
        const float off_a = mn_a == -INFINITY ? 0.f : mn_a, off_b = mn_b == -INFINITY ? 0.f : mn_b;
        const float corr_a = fast_exp2(m_a - off_a), corr_b = fast_exp2(m_b - off_b);   // 2^(-inf) = 0
        float sum_a = 0.f, sum_b = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            sc[j][e] = fast_exp2(sc[j][e] - off_a); sc[j][2 + e] = fast_exp2(sc[j][2 + e] - off_b);
            sum_a += sc[j][e]; sum_b += sc[j][2 + e];
          }
        }
        sum_a += __shfl_xor_sync(0xffffffffu, sum_a, 1); sum_a += __shfl_xor_sync(0xffffffffu, sum_a, 2);
        sum_b += __shfl_xor_sync(0xffffffffu, sum_b, 1); sum_b += __shfl_xor_sync(0xffffffffu, sum_b, 2);
        l_a = l_a * corr_a + sum_a; l_b = l_b * corr_b + sum_b;
        m_a = mn_a; m_b = mn_b;
        uint32_t pf[2][4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          pf[h][0] = pack_f16x2(sc[2 * h][0], sc[2 * h][1]); pf[h][1] = pack_f16x2(sc[2 * h][2], sc[2 * h][3]);
          pf[h][2] = pack_f16x2(sc[2 * h + 1][0], sc[2 * h + 1][1]); pf[h][3] = pack_f16x2(sc[2 * h + 1][2], sc[2 * h + 1][3]);
        }
        // V fragments: lane supplies the address of row (lane & 15) of a 16-position slice, column block (lane >> 4)
        const int v_row = sl0 + (lane & 15), v_pc = lane >> 4;
        // the running maxima often stay put: then the accumulators need no rescaling (one vote per warp)
        const bool rescale = !__all_sync(0xffffffffu, corr_a == 1.0f && corr_b == 1.0f);
#pragma unroll
        for (int nd = 0; nd < 16; nd += 2) {
          if (nd < ntiles) {
            if (rescale) {
              o[nd][0] *= corr_a; o[nd][1] *= corr_a; o[nd][2] *= corr_b; o[nd][3] *= corr_b;
              o[nd + 1][0] *= corr_a; o[nd + 1][1] *= corr_a; o[nd + 1][2] *= corr_b; o[nd + 1][3] *= corr_b;
            }
            uint32_t vf[4], vg[4];
            ldmatrix_x4_trans(vf, kv_addr(vs, v_row, nd + v_pc));
            ldmatrix_x4_trans(vg, kv_addr(vs, v_row + 16, nd + v_pc));
            mma_16816(o[nd], pf[0], vf[0], vf[1]);
            mma_16816(o[nd + 1], pf[0], vf[2], vf[3]);
            mma_16816(o[nd], pf[1], vg[0], vg[1]);
            mma_16816(o[nd + 1], pf[1], vg[2], vg[3]);
          }
        }
      }
    }
    if (tra && c == c_begin) tra[5] = globaltimer_ns();
    if (TMA) {
      // this warp is done with the buffer: hand it back to the loader (the unit's last one is kept for the merge)
      __syncwarp();
      if (c + 1 < c_end) { if (lane == 0) mbar_arrive(ctl->kv_empty + cur); }
      else hold_buf = cur;
    } else {
      epi_bar_sync();   // tile may be overwritten by the next chunk or unit
      if (P.att_dbl) cur ^= 1;
      else if (c + 1 < c_end) stage_issue(c + 1, 0, false);
    }
  }
  if (TMA) {
    // one verdict for all 128 threads (a wait may have run out in some of them only)
    if (!ok) ctl->abort_flag = 1;
    ok = group_ok(ctl, et);
    if (!ok) return;
    ks = ring + (size_t)hold_buf * kvbuf;   // every warp has finished reading it (the barriers above)
  } else {
    ks = kv0;   // (buffer 0 serves the merge below)
    if (!ok) return;
  }
  if (ps == 2) {
    // second half's state -> shared memory (the K/V tiles are free now) -> merged into the first's
    float4* mb = reinterpret_cast<float4*>(ks);
    const int ms = ntiles + 1;   // vectors per block: the output n-tiles, then (max, sum)
    if (active && part == 1) {
#pragma unroll
      for (int nd = 0; nd < 16; ++nd)
        if (nd < ntiles) mb[(mt * ms + nd) * 32 + lane] = make_float4(o[nd][0], o[nd][1], o[nd][2], o[nd][3]);
      mb[(mt * ms + ntiles) * 32 + lane] = make_float4(m_a, m_b, l_a, l_b);
    }
    epi_bar_sync();
    if (active && part == 0) {
      const float4 st = mb[(mt * ms + ntiles) * 32 + lane];
      const float M_a = fmaxf(m_a, st.x), M_b = fmaxf(m_b, st.y);
      const float off_a = M_a == -INFINITY ? 0.f : M_a, off_b = M_b == -INFINITY ? 0.f : M_b;
      const float wa = fast_exp2(m_a - off_a), wa2 = fast_exp2(st.x - off_a), wb = fast_exp2(m_b - off_b), wb2 = fast_exp2(st.y - off_b);
      l_a = l_a * wa + st.z * wa2; l_b = l_b * wb + st.w * wb2;
      m_a = M_a; m_b = M_b;
#pragma unroll
      for (int nd = 0; nd < 16; ++nd)
        if (nd < ntiles) {
          const float4 v = mb[(mt * ms + nd) * 32 + lane];
          o[nd][0] = o[nd][0] * wa + v.x * wa2; o[nd][1] = o[nd][1] * wa + v.y * wa2;
          o[nd][2] = o[nd][2] * wb + v.z * wb2; o[nd][3] = o[nd][3] * wb + v.w * wb2;
        }
    }
    // (copy path: the next unit's staging starts with a barrier of its own before it overwrites the tiles)
  }
  if (TMA) {
    // the merge buffer (the last chunk's tiles) goes back to the loader: one arrival per warp
    __syncwarp();
    if (lane == 0) mbar_arrive(ctl->kv_empty + hold_buf);
  }
  if (!active || part != 0) return;

  // write this warp's 16 rows straight from the accumulator fragments: the final output when the
  // unit saw every visible position, else the state (O, max, sum) for the merge that ends the phase
  if (a.n_ranges == 1) {
    const float ia = l_a > 0.f ? 1.0f / l_a : 0.f, ib = l_b > 0.f ? 1.0f / l_b : 0.f;
#pragma unroll
    for (int half_row = 0; half_row < 2; ++half_row) {
      const int ql = half_row ? ql_b : ql_a;
      if (ql < nQ) {
        const int q = q0 + ql;
        bf16* orow = P.o + (size_t)(a.off + q / G) * P.Hq * hd + (size_t)(kvh * G + q % G) * hd;
        const float inv = half_row ? ib : ia;
#pragma unroll
        for (int nd = 0; nd < 16; ++nd)
          if (nd < ntiles)
          {
            const float v0 = o[nd][2 * half_row] * inv, v1 = o[nd][2 * half_row + 1] * inv;
            const __nv_bfloat162 hi2 = __floats2bfloat162_rn(v0, v1);
            *reinterpret_cast<__nv_bfloat162*>(orow + nd * 8 + t4 * 2) = hi2;
            *reinterpret_cast<uint32_t*>(orow + (size_t)P.lo_row * P.Hq * hd + nd * 8 + t4 * 2) =
                pack_bf16x2(v0 - __low2float(hi2), v1 - __high2float(hi2));
          }
      }
    }
  } else {
#pragma unroll
    for (int half_row = 0; half_row < 2; ++half_row) {
      const int ql = half_row ? ql_b : ql_a;
      if (ql < nQ) {
        float* dst = P.attn_part + (size_t)part_set * P.attn_set_stride + ((size_t)part_slot * P.att_qblk + ql) * (hd + 4);
#pragma unroll
        for (int nd = 0; nd < 16; ++nd)
          if (nd < ntiles)
            *reinterpret_cast<float2*>(dst + nd * 8 + t4 * 2) = make_float2(o[nd][2 * half_row], o[nd][2 * half_row + 1]);
        if (t4 == 0) { dst[hd] = half_row ? m_b : m_a; dst[hd + 1] = half_row ? l_b : l_a; }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Attention unit on the 5th-generation tensor cores
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t smem_desc_sw128_ex(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffff) >> 4);
  d |= (uint64_t)(lbo >> 4) << 16;               // MN-major operands: distance between 64-element column blocks
  d |= (uint64_t)(sbo >> 4) << 32;               // distance between 8-row groups
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;                        // SWIZZLE_128B
  return d;
}
// Instruction descriptor: fp32 accumulator, fp16 A and B, A K-major, B K-major or MN-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc_f16(int n, int b_mn_major) {
  return (1u << 4) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// 16 consecutive fp32 columns of this thread's TMEM lane, written.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
        "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
        "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// One attention unit with both contractions on tcgen05 (head sizes 64 and 128, K/V chunks from the
// loader warp's ring).  The unit's up to 128 queries are the M rows: thread (TMEM lane) q owns query q.
// Per 64-position chunk:
//   S[q, j] = sum_d Q[q, d] K[j, d]   A = Q tile (K-major, swizzled, staged once per unit), B = the K chunk
//                                     as the bulk copies left it (K-major), accumulator S in TMEM;
//   every thread reads its row of S, applies the staircase mask, updates its running maximum and sum
//   (base 2) and writes its row of P = 2^(S - max) as fp16 into a swizzled P tile;
//   O[q, :] += sum_j P[q, j] V[j, :]  A = P tile, B = the V chunk as copied ([position][head dim]: MN-major
//                                     for the MMA, column blocks 8 KB apart, 8-row groups 1 KB apart),
//                                     accumulator O in TMEM across the unit's chunks.
// The MMAs are issued by the MMA warp's thread (attn_issue_tc below), which runs one chunk ahead: S of
// chunk c + 1 is computed while these threads work on chunk c (two S buffers in TMEM, two P tiles).
// When a running maximum moves, the warp rescales its rows of O in TMEM (load, multiply, store) after
// the previous P.V has completed and before it releases the P tile.  Rows past the unit's queries run
// along on zero queries.  This function is the compute group's side.
__device__ __noinline__ void attn_unit_tc(const Params& P, const Phase& ph, const AttnReq& a, int kvh, int range, int qblk, int part_slot, int part_set,
                                          uint8_t* att_smem, Ctl* ctl, int et, bool& ok, KvCons& kvc, const Waiter& W,
                                          uint32_t tmem_s, uint32_t tmem_o) {
  const int hd = P.hd, G = P.Hq / P.Hkv, nq = P.Hq * hd, halves = hd / 64;
  const int lane = et & 31, quad = ((et >> 5) + 2) & 3;       // compute warps are warps 2..5: TMEM lane quadrant = warp & 3
  const int ql = quad * 32 + lane;                             // this thread's query row (TMEM lane)
  const int Q = a.R * G;
  const int q0 = qblk * P.att_qblk, nQ = min(P.att_qblk, Q - q0);
  const int q_rows = P.att_q_rows;
  uint8_t* qs = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(att_smem) + 1023) & ~(uintptr_t)1023);   // halves x [q_rows][128 B]
  uint8_t* psm = qs + (size_t)halves * q_rows * 128;           // two P tiles of [q_rows][128 B]
  const int c_begin = range * a.cpu, c_end = min(a.n_chunks, c_begin + a.cpu);
  const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;

  // the unit's queries, swizzled: query index q -> row r = q / G, head = kvh * G + q % G; rows past nQ are zero.
  // (Every S MMA of the previous unit has completed: its chunks were all waited for.)
  {
    const int pieces = hd / 8;                                 // 16-byte pieces per query
    for (int it = et; it < q_rows * pieces; it += 128) {
      const int r = it / pieces, c = it % pieces;
      const bool on = r < nQ;
      const int q = on ? q0 + r : q0;
      cp_async16(qs + (size_t)(c >> 3) * q_rows * 128 + (size_t)r * 128 + (size_t)(((c & 7) ^ (r & 7)) << 4),
                 reinterpret_cast<const uint4*>(P.q16 + (size_t)(a.off + q / G) * nq + (size_t)(kvh * G + q % G) * hd) + c, on);
    }
    cp_async_commit();
    cp_async_wait_all();
    fence_proxy_async_smem();                                  // the tensor core reads these tiles through the async proxy
    __syncwarp();
    if (lane == 0) mbar_arrive(&ctl->q_full);
  }
  const bool mine = ql < nQ;
  const int last = mine ? a.base + (q0 + ql) / G : -1;         // last visible position of this thread's query
  float m_run = -INFINITY, l_run = 0.f;

  for (int c = c_begin; c < c_end && ok; ++c) {
    const uint32_t sb = kvc.sc & 1u, s_par = (kvc.sc >> 1) & 1u;
#ifdef STAIRS_TRACE
    unsigned long long* tl = (P.trace && blockIdx.x == 0 && et == 64 && kvc.sc < 300u) ? P.trace + (size_t)(2 + gridDim.x) * P.n_phases * 8 + 8000 + kvc.sc * 6 : nullptr;
    if (tl) tl[0] = (unsigned long long)clock64();
#endif
    ++kvc.sc;
    if (!W.wait(ctl->s_full + sb, s_par)) { ok = false; break; }   // S of chunk c is in TMEM
#ifdef STAIRS_TRACE
    if (tl) tl[1] = (unsigned long long)clock64();
#endif
    __syncwarp();
    tc_fence_after();
    const int p0 = c * ATT_CHUNK;
    const int n_pos = min(ATT_CHUNK, a.base + a.R - p0);
    const bool all_visible = p0 + ATT_CHUNK - 1 <= a.base;
    float sv[ATT_CHUNK];
#pragma unroll
    for (int j0 = 0; j0 < ATT_CHUNK; j0 += 16) tmem_ld16(tmem_s + sb * ATT_CHUNK + lane_sel + (uint32_t)j0, sv + j0);
#ifdef STAIRS_TRACE
    if (tl) tl[2] = (unsigned long long)clock64();
#endif
    if (!all_visible) {
#pragma unroll
      for (int j = 0; j < ATT_CHUNK; ++j)
        if (!(j < n_pos && p0 + j <= last)) sv[j] = -INFINITY;
    }
    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four independent chains
#pragma unroll
    for (int j = 0; j < ATT_CHUNK; j += 4) {
      mx4[0] = fmaxf(mx4[0], sv[j]); mx4[1] = fmaxf(mx4[1], sv[j + 1]); mx4[2] = fmaxf(mx4[2], sv[j + 2]); mx4[3] = fmaxf(mx4[3], sv[j + 3]);
    }
    const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
    // The reference exponent m_run only follows the running maximum when that has moved by more than
    // 2^8: until then P = 2^(S - m_run) may exceed 1 (at most 256: fine in fp16, and the sums are fp32),
    // and O needs no rescaling - the same reference scales O and the sum, so the quotient is unchanged.
    const float m_seen = fmaxf(m_run, mx);
    const float m_new = (m_seen > m_run + 8.0f || m_run == -INFINITY) ? m_seen : m_run;
    const float off = m_new == -INFINITY ? 0.f : m_new;
    const float corr = fast_exp2(m_run - off);                 // 1 when the reference stays; 2^(-inf) = 0
    float sum4[4] = {0.f, 0.f, 0.f, 0.f};
    uint32_t pk[ATT_CHUNK / 2];
#pragma unroll
    for (int j = 0; j < ATT_CHUNK; j += 2) {
      const float e0 = fast_exp2(sv[j] - off), e1 = fast_exp2(sv[j + 1] - off);
      sum4[(j >> 1) & 3] += e0 + e1;
      pk[j / 2] = pack_f16x2(e0, e1);
    }
    l_run = l_run * corr + ((sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));
    m_run = m_new;
    // the row of P: eight 16-byte pieces, swizzled like every K-major tile (the P.V that read this tile two
    // chunks ago has completed: the wait below covered it one chunk ago)
    if (ql < q_rows) {
      uint8_t* prow_s = psm + (size_t)sb * q_rows * 128 + (size_t)ql * 128;
#pragma unroll
      for (int cpc = 0; cpc < 8; ++cpc)
        *reinterpret_cast<uint4*>(prow_s + (size_t)((cpc ^ (ql & 7)) << 4)) = make_uint4(pk[4 * cpc], pk[4 * cpc + 1], pk[4 * cpc + 2], pk[4 * cpc + 3]);
    }
#ifdef STAIRS_TRACE
    if (tl) tl[3] = (unsigned long long)clock64();
#endif
    if (c > c_begin) {
      // the previous chunk's P.V has completed; O is rescaled where a maximum moved
      if (!W.wait(&ctl->o_done, kvc.o_par)) { ok = false; break; }
      kvc.o_par ^= 1u;
      __syncwarp();
      tc_fence_after();
      if (__any_sync(0xffffffffu, corr != 1.0f)) {
        for (int d0 = 0; d0 < hd; d0 += 16) {
          float ov[16];
          tmem_ld16(tmem_o + lane_sel + (uint32_t)d0, ov);
#pragma unroll
          for (int j = 0; j < 16; ++j) ov[j] *= corr;
          tmem_st16(tmem_o + lane_sel + (uint32_t)d0, ov);
        }
      }
    }
#ifdef STAIRS_TRACE
    if (tl) tl[4] = (unsigned long long)clock64();
#endif
    fence_proxy_async_smem();
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(ctl->p_full + sb);              // this warp's rows of P (and of O) are ready for the chunk's P.V
#ifdef STAIRS_TRACE
    if (tl) tl[5] = (unsigned long long)clock64();
#endif
  }
  // the unit's last P.V has completed
  if (ok) {
    if (!W.wait(&ctl->o_done, kvc.o_par)) ok = false;
    kvc.o_par ^= 1u;
  }
  __syncwarp();
  if (!ok) ctl->abort_flag = 1;
  ok = group_ok(ctl, et);                                      // one verdict for all 128 threads
  if (!ok) return;
  tc_fence_after();
  // this thread's row: the final output when the unit saw every visible position, else the state
  // (O, max, sum) for the merge that ends the phase.  (All lanes take part in the TMEM loads.)
  const int q = q0 + (mine ? ql : 0);
  const float inv = a.n_ranges == 1 ? (l_run > 0.f ? 1.0f / l_run : 0.f) : 1.0f;
  bf16* orow = P.o + (size_t)(a.off + q / G) * P.Hq * hd + (size_t)(kvh * G + q % G) * hd;
  float* prow = P.attn_part + (size_t)part_set * P.attn_set_stride + ((size_t)part_slot * P.att_qblk + (mine ? ql : 0)) * (hd + 4);
  for (int d0 = 0; d0 < hd; d0 += 16) {
    float ov[16];
    tmem_ld16(tmem_o + lane_sel + (uint32_t)d0, ov);
    if (mine) {
      if (a.n_ranges == 1) {
#pragma unroll
        for (int j = 0; j < 16; j += 4)
          store_split4(orow, (size_t)(d0 + j), (size_t)P.lo_row * P.Hq * hd, make_float4(ov[j] * inv, ov[j + 1] * inv, ov[j + 2] * inv, ov[j + 3] * inv));
      } else {
#pragma unroll
        for (int j = 0; j < 16; j += 4) *reinterpret_cast<float4*>(prow + d0 + j) = make_float4(ov[j], ov[j + 1], ov[j + 2], ov[j + 3]);
      }
    }
  }
  if (mine && a.n_ranges != 1) { prow[hd] = m_run; prow[hd + 1] = l_run; }
  tc_fence_before();
  // (the next unit's first P.V overwrites O only after these threads have released that unit's first P tile)
}

// The MMA warp's side of the tcgen05 attention: walks this CTA's units of one attention phase in the
// compute group's order and issues, per chunk, S = Q.K^T (as soon as the chunk's tiles have landed) and,
// one chunk behind, O += P.V (once the compute warps have released the P tile); a commit after each S
// signals the compute group, commits after each P.V hand the chunk buffer back to the loader and
// publish the completion.  mc: this thread's running state across phases.
struct AttIssue { int buf; uint32_t par; uint32_t sc; uint32_t q_par; };
__device__ __noinline__ bool attn_issue_tc(const Params& P, Ctl* ctl, uint8_t* att_smem, int cta, int G, const Waiter& W,
                                           uint32_t tmem_s, uint32_t tmem_o, AttIssue& mc) {
  const int hd = P.hd, halves = hd / 64, q_rows = P.att_q_rows;
  uint8_t* qs = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(att_smem) + 1023) & ~(uintptr_t)1023);
  uint8_t* psm = qs + (size_t)halves * q_rows * 128;
  uint8_t* ring = psm + (size_t)2 * q_rows * 128;
  const size_t kvbuf = AttnSmem::kv_buf_bytes(hd);
  const uint32_t idesc_s = instr_desc_f16(ATT_CHUNK, 0), idesc_o = instr_desc_f16(hd, 1);
  const int n_req = P.mode == CALL_VALIDATE ? P.n_req : 1;
  int u0 = 0;
  for (int i = 0; i < n_req; ++i) {
    const AttnReq a = ctl->areq[i];
    const int first = (cta - u0 % G + G) % G;
    for (int u = first; u < a.units; u += G) {
      const int rest = u / a.n_qblk;
      const int range = rest % a.n_ranges;
      const int c_begin = range * a.cpu, c_end = min(a.n_chunks, c_begin + a.cpu);
      if (!W.wait(&ctl->q_full, mc.q_par)) return false;      // the unit's Q tile is staged
      mc.q_par ^= 1u;
      // Two streams of work, each issued as soon as its input is there: S of the next chunk (its tiles
      // have landed; at most one chunk ahead of the P.V stream, because there are two S buffers) and
      // P.V of the oldest chunk whose P tile the compute warps have released.  Taking whichever is
      // ready keeps a late chunk from holding up the P.V that frees a buffer for the loader.
      int s_next = c_begin, pv_next = c_begin;
      int pv_buf = mc.buf; uint32_t pv_n = mc.sc;              // buffer and running chunk number of the next P.V
      long long t_idle = 0; bool idle = false;
      while (pv_next < c_end) {
        bool progress = false;
        if (s_next < c_end && s_next - pv_next <= 1 && mbar_test(ctl->kv_full + mc.buf, mc.par)) {
          tc_fence_after();
          const uint32_t sb = mc.sc & 1u;
          const uint32_t kb = smem_u32(ring + (size_t)mc.buf * kvbuf);
          for (int h = 0; h < halves; ++h)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              umma_bf16(tmem_s + sb * ATT_CHUNK, smem_desc_sw128_ex(smem_u32(qs) + (uint32_t)(h * q_rows * 128 + k * 32), 16, 1024),
                        smem_desc_sw128_ex(kb + (uint32_t)(h * ATT_CHUNK * 128 + k * 32), 16, 1024), idesc_s, (h | k) ? 1u : 0u);
          umma_commit(ctl->s_full + sb);
          ++mc.sc; ++s_next;
          if (++mc.buf == P.att_nbuf) { mc.buf = 0; mc.par ^= 1u; }
          progress = true;
        }
        if (pv_next < s_next && mbar_test(ctl->p_full + (pv_n & 1u), (pv_n >> 1) & 1u)) {
          tc_fence_after();
          const uint32_t vb = smem_u32(ring + (size_t)pv_buf * kvbuf + kvbuf / 2);
          const uint32_t pb = smem_u32(psm + (size_t)(pv_n & 1u) * q_rows * 128);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_bf16(tmem_o, smem_desc_sw128_ex(pb + (uint32_t)(k * 32), 16, 1024),
                      smem_desc_sw128_ex(vb + (uint32_t)(k * 2048), (uint32_t)(ATT_CHUNK * 128), 1024), idesc_o, (pv_next > c_begin || k > 0) ? 1u : 0u);
          umma_commit(ctl->kv_empty + pv_buf);
          umma_commit(&ctl->o_done);
          ++pv_n; ++pv_next;
          if (++pv_buf == P.att_nbuf) pv_buf = 0;
          progress = true;
        }
        if (progress) idle = false;
        else {
          if (!idle) { idle = true; t_idle = clock64(); }
          if (W.poll_abort(t_idle)) { W.note(5u, (unsigned)cta, (unsigned)s_next, (unsigned)pv_next, (unsigned)mc.sc); return false; }
        }
      }
    }
    u0 += a.units;
  }
  return true;
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(MK_THREADS, 1) k_forward(const __grid_constant__ Params P) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int stages = P.stages;
  const int kps = P.kps;
  const int a_stage_bytes = kps * A_STAGE_BYTES;            // kps weight slabs of 128 rows x 128 bytes
  const int b_kb_bytes = 2 * P.t_box * BK * 2;              // activation slab of one k-block: hi rows then lo rows
  const int stage_bytes = a_stage_bytes + kps * b_kb_bytes;
  uint8_t* tail = smem + (size_t)stages * stage_bytes;
  float* vt = reinterpret_cast<float*>(tail);   // epilogue exchange tile [16][VT_LD]
  Ctl* ctl = reinterpret_cast<Ctl*>(tail + MK_XCH_BYTES);
  uint8_t* att_smem = tail + MK_XCH_BYTES + ((sizeof(Ctl) + 127) & ~(size_t)127);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = gridDim.x, cta = blockIdx.x;
  uint32_t tmem_cols = 32;
  // two GEMM accumulators, each with hi-part and lo-part columns; tcgen05 attention adds S (one chunk) and O (head size)
  const uint32_t tmem_att = (uint32_t)(4 * P.t_box);
  while ((int)tmem_cols < 4 * P.t_box + (P.att_tc ? 2 * ATT_CHUNK + P.hd : 0)) tmem_cols <<= 1;   // two S buffers, O

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(ctl->full + s, 1); mbar_init(ctl->empty + s, 1); }
    mbar_init(ctl->acc_full + 0, 1); mbar_init(ctl->acc_full + 1, 1);
    mbar_init(ctl->acc_empty + 0, 4); mbar_init(ctl->acc_empty + 1, 4);
    // a chunk buffer is handed back by the four compute warps (mma.sync path) or by one tcgen05.commit
    for (int b = 0; b < MAX_KV_BUF; ++b) { mbar_init(ctl->kv_full + b, 1); mbar_init(ctl->kv_empty + b, P.att_tc ? 1 : 4); }
    mbar_init(ctl->s_full + 0, 1); mbar_init(ctl->s_full + 1, 1);
    mbar_init(ctl->p_full + 0, 4); mbar_init(ctl->p_full + 1, 4);
    mbar_init(&ctl->q_full, 4); mbar_init(&ctl->o_done, 1);
    ctl->abort_flag = 0; ctl->bcast = 0; ctl->areq_ready = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(&ctl->tmem_slot, tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_slot;
  const Waiter W{&ctl->abort_flag, P.bar + 1, P.wait_limit, P.status};
  const unsigned long long* bar_count = P.bar;
  // producer bookkeeping for the abort path
  int issued = 0, p_stage = 0;
  uint32_t p_phase = 0;

  if (warp == 0) {
    // ================================================================== TMA producer
    if (lane == 0) {
      const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
      WCursor A, B;
      A.enter(P, cta, G, 0); B.enter(P, cta, G, 0);
      int a_stage = 0, b_stage = 0;
      uint32_t a_par = 0;
      unsigned int a_count = 0, b_count = 0, idle = 0;
      int ready_ph = -1;   // phases <= ready_ph have their inputs published
      unsigned long long poll_val = 0; bool poll_pending = false;
      int traced_ph = -1;
      long long t_idle = clock64();
      while (B.valid) {
        bool progress = false;
        if (A.valid && mbar_test(ctl->empty + a_stage, a_par ^ 1)) {
          uint8_t* a_dst = smem + (size_t)a_stage * stage_bytes;
          mbar_expect_tx(ctl->full + a_stage, (uint32_t)stage_bytes);
          tma_load_3d(a_dst, A.wm0, 0, A.row, A.kk * kps, ctl->full + a_stage, pol_w);
#ifdef STAIRS_TRACE
          if (P.trace && cta == 0) P.trace[(size_t)(2 + G) * P.n_phases * 8 + 4000 + a_count] = (unsigned long long)clock64();
#endif
          ++issued; ++a_count;
          if (++a_stage == stages) { a_stage = 0; a_par ^= 1; }
          p_stage = a_stage; p_phase = a_par;
          A.advance(P, cta, G);
          progress = true;
        }
        if (b_count != a_count) {
          // Inputs of phase B.ph are published once every CTA has finished phase B.ph - 1.  The
          // poll is a global acquire load (a long round trip): it is issued in one pass of this
          // loop and looked at in the next, so that weight tiles keep being issued under it.
          if (B.ph > ready_ph) {
            if (poll_pending && poll_val >= P.bar_base + (unsigned long long)B.ph * G) { ready_ph = B.ph; fence_proxy_async(); }
            poll_pending = false;
            if (B.ph > ready_ph) { poll_val = ld_acquire_u64(bar_count); poll_pending = true; }
          }
          if (B.ph <= ready_ph) {
            uint8_t* b_dst = smem + (size_t)b_stage * stage_bytes + a_stage_bytes;
            tma_load_3d(b_dst, P.maps + B.x_map, 0, 0, B.kk * kps, ctl->full + b_stage, pol_x);   // hi and lo rows in one box
            if (MK_TRACE_PTR(P.trace) && cta == 0 && B.ph != traced_ph) { traced_ph = B.ph; MK_TRACE_PTR(P.trace)[(size_t)B.ph * 8 + 7] = globaltimer_ns(); }
#ifdef STAIRS_TRACE
            if (P.trace && cta == 0) P.trace[(size_t)(2 + G) * P.n_phases * 8 + 6000 + b_count] = (unsigned long long)clock64();
#endif
            ++b_count;
            if (++b_stage == stages) b_stage = 0;
            B.advance(P, cta, G);
            progress = true;
          }
        }
        if (progress) idle = 0;
        else {
          if (idle++ == 0) t_idle = clock64();   // (the clock is only read once the producer goes idle)
          if (W.poll_abort(t_idle)) break;
          if ((idle & 4095u) == 0 && ld_acquire_u64(P.bar + 1)) { ctl->abort_flag = 1; break; }
        }
      }
    }
  } else if (warp == 1) {
    // ================================================================== MMA issuer
    if (lane == 0) {
      // One MMA covers the hi and the lo rows of the activation tile (they are adjacent in the
      // stage: N = 2 * t_box); the two halves of the accumulator are added when it is drained.
      const uint32_t idesc = instr_desc_bf16(2 * P.t_box);
      int stage = 0; uint32_t phase = 0;
      int buf = 0; uint32_t acc_bits = 0;   // bit b: parity of accumulator b (no run-time indexed array: see the cursor)
      bool ok = true;
#ifdef STAIRS_TRACE
      unsigned long long* klog = P.trace ? P.trace + (size_t)(2 + G) * P.n_phases * 8 : nullptr;   // per k-block cycle stamps of CTA 0
      int kn = 0;
#endif
      AttIssue att_mc{0, 0u, 0u, 0u};
      bool areq_seen = false;
      for (int ph = 0; ph < P.n_phases && ok; ++ph) {
        const Phase& p = P.phases[ph];
        if (p.kind == PH_ATTN && P.att_tc) {
          // attention contractions of this CTA's units (the compute group does the softmax in between)
          if (!areq_seen) {
            const long long t0 = clock64();
            while (!(areq_seen = ctl->areq_ready != 0)) { if (W.poll_abort(t0)) break; }
            if (!areq_seen) { ok = false; break; }
          }
          ok = attn_issue_tc(P, ctl, att_smem, cta, G, W, tmem_base + tmem_att, tmem_base + tmem_att + 2 * ATT_CHUNK, att_mc);
          continue;
        }
        if (p.kind != PH_GEMM) continue;
        const int kblocks = p.kblocks;
        const KRange kr = phase_range(p.n_tiles, p.upt, kblocks, RANGE_UNIT_KB / kps, cta, G, p.ge_max);
        int remaining = kr.end - kr.begin;
        if (remaining <= 0) continue;
        int kk = kr.begin % kblocks;
        bool seg_first = true;
        unsigned long long* trm = (MK_TRACE_PTR(P.trace) && cta == 0) ? MK_TRACE_PTR(P.trace) + (size_t)ph * 8 : nullptr;
        bool first_k = true;
        while (remaining > 0 && ok) {
          const bool seg_last = (remaining == 1) || (kk == kblocks - 1);
          if (seg_first) {
            ok = W.wait(ctl->acc_empty + buf, ((acc_bits >> buf) & 1u) ^ 1u);
            if (!ok) break;
            tc_fence_after();
          }
#ifdef STAIRS_TRACE
          if (trm) klog[3 * kn] = (unsigned long long)clock64();
#endif
          ok = W.wait(ctl->full + stage, phase);
          if (!ok) break;
          if (trm && first_k) { trm[5] = globaltimer_ns(); first_k = false; }
#ifdef STAIRS_TRACE
          if (trm) klog[3 * kn + 1] = (unsigned long long)clock64();
#endif
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + (size_t)stage * stage_bytes);
          const uint64_t a_desc = smem_desc_sw128(a_addr), b_desc = smem_desc_sw128(a_addr + (uint32_t)a_stage_bytes);
          const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 2 * P.t_box);
          // every k-block of the stage (a k-block past the end of K was zero-filled by the copies)
          for (int j = 0; j < kps; ++j) {
            const uint64_t aj = a_desc + (uint64_t)((j * A_STAGE_BYTES) >> 4), bj = b_desc + (uint64_t)((j * b_kb_bytes) >> 4);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k)
              umma_bf16(d_tmem, aj + (uint64_t)(k * UMMA_K * 2 / 16), bj + (uint64_t)(k * UMMA_K * 2 / 16), idesc,
                        (seg_first && j == 0 && k == 0) ? 0u : 1u);
          }
          // (a commit costs about 240 cycles of issue time: the one the epilogue waits for goes first)
          if (seg_last) { umma_commit(ctl->acc_full + buf); acc_bits ^= 1u << buf; buf ^= 1; }
          umma_commit(ctl->empty + stage);
#ifdef STAIRS_TRACE
          if (trm) { klog[3 * kn + 2] = (unsigned long long)clock64(); ++kn; }
#endif
          seg_first = seg_last;
          if (++kk == kblocks) kk = 0;
          --remaining;
          if (++stage == stages) { stage = 0; phase ^= 1; }
        }
        if (trm) trm[6] = globaltimer_ns();
      }
    }
  } else if (warp == 6) {
    // ================================================================== K/V loader of the attention phases (TMA path)
    // Walks this CTA's attention units of every attention phase in the compute group's order and
    // streams their K/V chunks through the ring of chunk buffers: per chunk one box per (K or V,
    // 64-column half, page slice), each issued by its own lane.  Chunks that hold only positions
    // cached by earlier calls are fetched as soon as a buffer is free - also ahead of the phase;
    // a chunk with positions of this call waits for the grid barrier that publishes them.
    if (P.att_tma) {
      bool ok = true;
      {
        bool seen = false;
        if (lane == 0) {
          const long long t0 = clock64();
          while (!(seen = ctl->areq_ready != 0)) { if (W.poll_abort(t0)) break; }
        }
        ok = __shfl_sync(0xffffffffu, seen ? 1 : 0, 0) != 0;
        __syncwarp();
      }
      const int hd = P.hd, halves = hd / 64, box_rows = P.kv_box_rows, slots = ATT_CHUNK / box_rows;
      const int n_boxes = 2 * halves * slots;
      const size_t kvbuf = AttnSmem::kv_buf_bytes(hd);
      uint8_t* ring = att_ring_base(P, att_smem);
      // this lane's box: which tensor (K, V), which 64-column half, which page slice of the chunk
      const int b_which = lane / (halves * slots), b_half = (lane % (halves * slots)) / slots, b_slot = lane % slots;
      int buf = 0; uint32_t par = 0;
      uint32_t used = 0, last_par = 0;   // per buffer: ever filled, and the parity of its latest fill
      const int n_req = P.mode == CALL_VALIDATE ? P.n_req : 1;
      for (int ph = 0; ph < P.n_phases && ok; ++ph) {
        const Phase& p = P.phases[ph];
        if (p.kind != PH_ATTN) continue;
        const CUtensorMap* kmap = P.maps + p.w_map[0];
        const CUtensorMap* vmap = P.maps + p.w_map[1];
        bool published = false;   // the grid barrier before this phase has completed
        int u0 = 0;
        for (int i = 0; i < n_req && ok; ++i) {
          const AttnReq a = ctl->areq[i];
          const int* pt = P.page_table + (size_t)a.slot * P.max_pages;
          const int first = (cta - u0 % G + G) % G;
          for (int u = first; u < a.units && ok; u += G) {
            const int rest = u / a.n_qblk;
            const int range = rest % a.n_ranges, kvh = rest / a.n_ranges;
            const int c_begin = range * a.cpu, c_end = min(a.n_chunks, c_begin + a.cpu);
            for (int c = c_begin; c < c_end && ok; ++c) {
              const int p0 = c * ATT_CHUNK;
              // page slices of the chunk inside the request's page table (the rest keeps its old, finite contents);
              // this lane's cache row is looked up before the wait for a free buffer, under which its latency hides
              const int valid_slots = min(slots, (P.max_pages * P.page_tokens - p0) / box_rows);
              const bool my_box = lane < n_boxes && b_slot < valid_slots;
              const int pz = p0 + b_slot * box_rows;
              const int row = my_box ? __ldcg(pt + pz / P.page_tokens) * P.page_tokens + pz % P.page_tokens : 0;
              bool go = true;
              if (lane == 0) {
                if (p0 + ATT_CHUNK > a.base && !published) go = W.wait_grid(bar_count, P.bar_base + (unsigned long long)ph * G);
                if (go) go = W.wait(ctl->kv_empty + buf, par ^ 1u);
              }
              ok = __shfl_sync(0xffffffffu, go ? 1 : 0, 0) != 0;
              if (!ok) break;
              if (p0 + ATT_CHUNK > a.base && !published) { published = true; fence_proxy_async(); }
              if (lane == 0) mbar_expect_tx(ctl->kv_full + buf, (uint32_t)(2 * halves * valid_slots * box_rows * 128));
              __syncwarp();
              if (my_box) {
                uint8_t* dst = ring + (size_t)buf * kvbuf + (size_t)b_which * (kvbuf / 2) + (size_t)b_half * (ATT_CHUNK * 128) + (size_t)b_slot * box_rows * 128;
                tma_load_2d_nohint(dst, b_which ? vmap : kmap, kvh * hd + b_half * 64, row, ctl->kv_full + buf);
              }
              __syncwarp();
              used |= 1u << buf;
              last_par = (last_par & ~(1u << buf)) | (par << buf);
              if (++buf == P.att_nbuf) { buf = 0; par ^= 1u; }
            }
          }
          u0 += a.units;
        }
      }
      // After an abort copies may still be in flight: they must land before the CTA's shared memory
      // is given up (bounded, like the producer's drain below; after a healthy pass every fill
      // was consumed, so these tests succeed at once).
      if (lane == 0) {
        const long long t0 = clock64();
        const unsigned long long drain_limit = P.wait_limit > 2000000ull ? P.wait_limit : 2000000ull;
        for (int b = 0; b < P.att_nbuf; ++b)
          if (used & (1u << b))
            while (!mbar_try(ctl->kv_full + b, (last_par >> b) & 1u)) {
              if ((unsigned long long)(clock64() - t0) > drain_limit) break;
            }
      }
    }
  } else {
    // ================================================================== compute group (warps 2..5)
    const int quad = warp & 3;
    const int m = quad * 32 + lane;
    const int et = threadIdx.x - 64;
    float* red = vt;    // 4 floats of scratch for group sums (the exchange tile is free outside GEMM epilogues)
    int buf = 0; uint32_t acc_bits = 0;
    bool ok = true;
    bool waited = true;   // true when every earlier phase is known complete grid-wide

    constexpr int PH_WORDS = (int)((sizeof(Phase) + 3) / 4);
    static_assert(PH_WORDS <= 128, "one descriptor word per compute thread");
    {
      // descriptor of phase 0 and the requests' attention geometry, once
      if (et < PH_WORDS) ctl->phc[0][et] = __ldcg(reinterpret_cast<const uint32_t*>(P.phases) + et);
      const int n_req0 = P.mode == CALL_VALIDATE ? P.n_req : 1;
      if (et < n_req0 && et < 64) ctl->areq[et] = attn_req(P, et, G);
      if (P.att_tma) {
        // the chunk buffers start out finite: a box that is never fetched (past the page table) must not feed NaNs to P.V
        uint8_t* ring = att_ring_base(P, att_smem);
        uint8_t* first = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(att_smem) + 1023) & ~(uintptr_t)1023);   // (the Q and P tiles too)
        const int n16 = (int)((size_t)(ring - first) + (size_t)P.att_nbuf * AttnSmem::kv_buf_bytes(P.hd)) / 16;
        for (int i = et; i < n16; i += 128) reinterpret_cast<uint4*>(first)[i] = make_uint4(0u, 0u, 0u, 0u);
        fence_proxy_async_smem();   // later bulk copies (async proxy) into these buffers
      }
      epi_bar_sync();
      if (et == 0) { __threadfence_block(); ctl->areq_ready = 1; }
    }
    KvCons kvc{0, 0u, 0u, 0u};
    // Split-tile partial sums: two sets of slots, used by alternate GEMM phases; the slots a finisher
    // has read are emptied again one GEMM phase later (or at the end of the kernel), while it waits
    // for that phase's accumulator - off the chain that ends a phase, and before the set's next use.
    int gph = 0;                               // GEMM phases so far
    unsigned pend_first = 1u, pend_last = 0u;  // slots (CTAs) read and not yet emptied
    int pend_set = 0;
    auto slot_of = [&](int set, unsigned c) { return P.partial + ((size_t)set * G + c) * P.t_box * BM; };
    auto empty_pending = [&]() {
      const int er_ = et >> 3, cg_ = et & 7;
      for (unsigned c = pend_first; c <= pend_last; ++c)
        for (int t = er_; t < P.T; t += 16) {
          float* row = slot_of(pend_set, c) + (size_t)t * BM;
#pragma unroll
          for (int q = 0; q < 4; ++q) st_relaxed_u4(row + (cg_ + 8 * q) * 4, make_uint4(PARTIAL_EMPTY, PARTIAL_EMPTY, PARTIAL_EMPTY, PARTIAL_EMPTY));
        }
      pend_first = 1u; pend_last = 0u;
    };
    // Parked attention states: two sets, used by alternate attention phases.  The states are merged
    // inside the attention phase itself (each warp polls the words it needs: no grid barrier in
    // between); a CTA empties the slots of its own units one attention phase later, while it waits
    // for that phase's inputs, and those of the last phase at the end of the kernel.
    int aph = 0;   // attention phases so far
    auto empty_own_states = [&](int set) {
      const int n_req_ = P.mode == CALL_VALIDATE ? P.n_req : 1;
      const int Gq_ = P.Hq / P.Hkv, row_words = P.hd + 4;
      int u0_ = 0;
      for (int i = 0; i < n_req_; ++i) {
        const AttnReq a = ctl->areq[i];
        if (a.n_ranges > 1) {
          const int first = (cta - u0_ % G + G) % G;
          for (int u = first; u < a.units; u += G) {
            const int qblk = u % a.n_qblk;
            const int nQ = min(P.att_qblk, a.R * Gq_ - qblk * P.att_qblk);
            if (u0_ + u >= P.attn_part_units) break;
            float* st = P.attn_part + (size_t)set * P.attn_set_stride + (size_t)(u0_ + u) * P.att_qblk * row_words;
            for (int w4 = et; w4 < nQ * row_words / 4; w4 += 128)
              st_relaxed_u4(st + w4 * 4, make_uint4(PARTIAL_EMPTY, PARTIAL_EMPTY, PARTIAL_EMPTY, PARTIAL_EMPTY));
          }
        }
        u0_ += a.units;
      }
    };
    for (int ph = 0; ph < P.n_phases && ok; ++ph) {
      const Phase& p = *reinterpret_cast<const Phase*>(ctl->phc[ph & 1]);
      if (p.kind == PH_ATTN && aph > 0) empty_own_states((aph & 1) ^ 1);   // (read by the previous attention phase, which every CTA has left)
      // the next phase's descriptor: fetched now, parked in shared memory at the end of this phase
      const uint32_t next_word = (et < PH_WORDS && ph + 1 < P.n_phases) ? __ldcg(reinterpret_cast<const uint32_t*>(P.phases + ph + 1) + et) : 0u;
      if (p.kind != PH_GEMM && !waited) {
        // inputs come from other CTAs: wait until all of them finished phase ph - 1
        if (et == 0) {
          const bool g = W.wait_grid(bar_count, P.bar_base + (unsigned long long)ph * G);
          ctl->bcast = g ? 1 : 0;
        }
        epi_bar_sync();
        ok = ctl->bcast != 0;
        epi_bar_sync();
        if (!ok) break;
      }

      bool gemm_worked = false;
      const bool tracing = MK_TRACE_PTR(P.trace) && et == 0 && (cta == 0 || cta == G - 1);
      unsigned long long* tr = tracing ? MK_TRACE_PTR(P.trace) + ((size_t)(cta == 0 ? 0 : 1) * P.n_phases + ph) * 8 : nullptr;
      if (tracing) tr[0] = globaltimer_ns();
      if (p.kind == PH_EMBED) {
        if (cta == 0)
          for (int i = et; i < P.n_keys; i += 128) P.keys[i] = 0ull;
        for (int t = cta; t < P.T; t += G) {
          const RowInfo r = row_info(P, t);
          if (et == 0) { P.tok[t] = r.tok; P.pos[t] = r.pos; P.req[t] = r.slot; }
          embed_row(P, t, r, p.g, red, et);
        }
      } else if (p.kind == PH_ATTN) {
        const int n_req = P.mode == CALL_VALIDATE ? P.n_req : 1;
        int u0 = 0, g0 = 0;
        for (int i = 0; i < n_req && ok; ++i) {
          const AttnReq a = ctl->areq[i];
          // units of this request: index = ((kvh * n_ranges) + range) * n_qblk + qblk
          int first = (cta - u0 % G + G) % G;
          for (int u = first; u < a.units && ok; u += G) {
            const int qblk = u % a.n_qblk, rest = u / a.n_qblk;
            const int range = rest % a.n_ranges, kvh = rest / a.n_ranges;
            const int slot = u0 + u;
            if (slot >= P.attn_part_units) {
              // cannot happen while the host's bound holds; never compute part of a call silently
              if (et == 0) { W.note(4u, (unsigned)slot, (unsigned)P.attn_part_units, (unsigned)i, (unsigned)u); ctl->abort_flag = 1; }
              ok = group_ok(ctl, et);
              break;
            }
            unsigned long long* tra_u = (MK_TRACE_PTR(P.trace) && et == 0 && u == first) ? MK_TRACE_PTR(P.trace) + (size_t)2 * P.n_phases * 8 + ((size_t)cta * P.n_phases + ph) * 8 : nullptr;
            if (P.att_tc) attn_unit_tc(P, p, a, kvh, range, qblk, slot, aph & 1, att_smem, ctl, et, ok, kvc, W, tmem_base + tmem_att, tmem_base + tmem_att + 2 * ATT_CHUNK);
            else if (P.att_tma) attn_unit<true>(P, p, a, kvh, range, qblk, slot, aph & 1, att_smem, ctl, et, ok, kvc, W, tra_u);
            else attn_unit<false>(P, p, a, kvh, range, qblk, slot, aph & 1, att_smem, ctl, et, ok, kvc, W, tra_u);
          }
          u0 += a.units; g0 += P.Hkv * a.n_qblk;
        }
        // Requests whose positions were split over several units: merge the parked states of every
        // (kv head, query) in position order.  One warp per item; each lane owns 4 consecutive
        // elements of head_dim, so every partial is one 16-byte load per lane.  The states come
        // from other CTAs' units of this same phase: a word reads PARTIAL_EMPTY until it has been
        // stored, and the warp repeats its loads (bounded) until none does.
        if (ok) {
          const int hd = P.hd, Gq = P.Hq / P.Hkv;
          const float* set_base = P.attn_part + (size_t)(aph & 1) * P.attn_set_stride;
          int u0c = 0, item0 = 0;
          bool gave_up = false;
          auto backoff = [&](long long& t0, bool& timing) {   // warp-uniform: true when the wait has run out
            if (!timing) { t0 = clock64(); timing = true; }
            bool quit = false;
            if (lane == 0) quit = W.poll_abort(t0);
            quit = __shfl_sync(0xffffffffu, quit ? 1 : 0, 0) != 0;
            if (quit && lane == 0) W.note(5u, (unsigned)ph, (unsigned)cta, 0u, 0u);
            if (!quit) __nanosleep(64);
            return quit;
          };
          for (int i = 0; i < n_req; ++i) {
            const AttnReq a = ctl->areq[i];
            if (a.n_ranges > 1) {
              const int Q = a.R * Gq, items = P.Hkv * Q;
              int it = ((cta * 4 + quad) - item0) % (G * 4);
              if (it < 0) it += G * 4;
              for (; it < items && !gave_up; it += G * 4) {
                const int kvh = it / Q, q = it % Q, qblk = q / P.att_qblk, ql = q % P.att_qblk;
                const int first_slot = u0c + (kvh * a.n_ranges) * a.n_qblk + qblk;
                const size_t stride = (size_t)a.n_qblk * P.att_qblk * (hd + 4);
                const float* base = set_base + ((size_t)first_slot * P.att_qblk + ql) * (hd + 4);
                // (max, sum) of range lane, lane + 32, ...: one load round for up to 32 ranges, then
                // the ranges' output vectors eight loads at a time; weights travel by shuffle and
                // the accumulation stays in range order
                const int nr = a.n_ranges, dd = lane * 4;
                long long t0 = 0;
                bool timing = false;
                auto state_of = [&](int r, float& mu, float& lu) {   // all lanes call it together
                  mu = -INFINITY; lu = 0.f;
                  while (true) {
                    uint2 v = make_uint2(0u, 0u);
                    if (r < nr) v = ld_relaxed_u2(base + r * stride + hd);
                    if (!__any_sync(0xffffffffu, v.x == PARTIAL_EMPTY || v.y == PARTIAL_EMPTY)) {
                      if (r < nr) { mu = __uint_as_float(v.x); lu = __uint_as_float(v.y); }
                      return;
                    }
                    if (backoff(t0, timing)) { gave_up = true; return; }
                  }
                };
                float M = -INFINITY, m0 = -INFINITY, l0 = 0.f;
                for (int rb = 0; rb < nr && !gave_up; rb += 32) {
                  float mu, lu;
                  state_of(rb + lane, mu, lu);
                  if (rb == 0) { m0 = mu; l0 = lu; }
                  M = fmaxf(M, mu);
                }
                M = warp_max(M);
                float L = 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int rb = 0; rb < nr && !gave_up; rb += 32) {
                  float mu = m0, lu = l0;
                  if (rb != 0) state_of(rb + lane, mu, lu);
                  const float wgt = mu == -INFINITY ? 0.f : fast_exp2(mu - M);   // 0 for lanes past the last range (maxima are base-2 exponents)
                  L += lu * wgt;
                  const int nb = min(32, nr - rb);
                  for (int g0 = 0; g0 < nb && !gave_up; g0 += 8) {
                    uint4 v[8];
                    while (true) {
                      uint32_t mx = 0u;
#pragma unroll
                      for (int u = 0; u < 8; ++u) {
                        v[u] = (g0 + u < nb && dd < hd) ? ld_relaxed_u4(base + (size_t)(rb + g0 + u) * stride + dd) : make_uint4(0u, 0u, 0u, 0u);
                        mx = max(max(mx, max(v[u].x, v[u].y)), max(v[u].z, v[u].w));
                      }
                      if (!__any_sync(0xffffffffu, mx == PARTIAL_EMPTY)) break;
                      if (backoff(t0, timing)) { gave_up = true; break; }
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                      const float wu = __shfl_sync(0xffffffffu, wgt, (g0 + u) & 31);
                      acc.x += __uint_as_float(v[u].x) * wu; acc.y += __uint_as_float(v[u].y) * wu;
                      acc.z += __uint_as_float(v[u].z) * wu; acc.w += __uint_as_float(v[u].w) * wu;
                    }
                  }
                }
                L = warp_sum(L);
                if (dd < hd) {
                  bf16* orow = P.o + (size_t)(a.off + q / Gq) * P.Hq * hd + (size_t)(kvh * Gq + q % Gq) * hd + dd;
                  const float inv = 1.0f / L;
                  const __nv_bfloat162 h01 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), h23 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
                  *reinterpret_cast<uint2*>(orow) = make_uint2(*reinterpret_cast<const uint32_t*>(&h01), *reinterpret_cast<const uint32_t*>(&h23));
                  *reinterpret_cast<uint2*>(orow + (size_t)P.lo_row * P.Hq * hd) =
                      make_uint2(pack_bf16x2(acc.x * inv - __low2float(h01), acc.y * inv - __high2float(h01)),
                                 pack_bf16x2(acc.z * inv - __low2float(h23), acc.w * inv - __high2float(h23)));
                }
              }
              item0 += items;
            }
            u0c += a.units;
          }
        }
        ++aph;
      } else if (p.kind == PH_PREP) {
        // Models whose head size is neither 64 nor 128: a rotation pair (i, i + hd/2) need not sit in
        // one thread (or one tile) of the QKV epilogue, so that epilogue stores fp32 and this extra
        // phase rotates, converts and files q, k and v.  One item = one pair of one head of one row.
        const int hd = P.hd, half = hd / 2, nq = P.Hq * hd, nkv = P.Hkv * hd, nqkv = nq + 2 * nkv, heads = P.Hq + 2 * P.Hkv;
        const int items = P.T * heads * half;
        const float qscale = 1.4426950408889634f / sqrtf((float)hd);   // log2(e) / sqrt(hd): the softmax works in base 2
        for (int it = cta * 128 + et; it < items; it += G * 128) {
          const int i = it % half, hs = (it / half) % heads, t = it / (half * heads);
          const float* row = P.qkv + (size_t)t * nqkv + (size_t)hs * hd;   // q heads, then k heads, then v heads
          float x0 = __ldcg(row + i), x1 = __ldcg(row + i + half);
          if (P.rope && hs < P.Hq + P.Hkv) {
            const float cs = __ldcg(P.rope_cs + (size_t)t * half + i), sn = __ldcg(P.rope_sn + (size_t)t * half + i);
            const float r0 = x0 * cs - x1 * sn, r1 = x1 * cs + x0 * sn;
            x0 = r0; x1 = r1;
          }
          if (hs < P.Hq) {
            __half* dst = P.q16 + (size_t)t * nq + (size_t)hs * hd;
            dst[i] = __float2half_rn(x0 * qscale); dst[i + half] = __float2half_rn(x1 * qscale);
          } else {
            const bool is_k = hs < P.Hq + P.Hkv;
            __half* dst = reinterpret_cast<__half*>(is_k ? p.kc : p.vc) + (size_t)cache_row_of(P, t) * nkv +
                          (size_t)(hs - P.Hq - (is_k ? 0 : P.Hkv)) * hd;
            dst[i] = __float2half_rn(x0); dst[i + half] = __float2half_rn(x1);
          }
        }
      } else if (p.kind == PH_ACCEPT) {
        if (cta == 0) {
          if (P.mode == CALL_VALIDATE) {
            for (int i = et; i < P.n_req; i += 128) {
              const int k = P.val_k[i], off = P.val_off[i], slot = P.val_req[i];
              int a = -1;
              for (int r = 0; r <= k; ++r) {
                const int tr = argmax_key_index(__ldcg(P.keys + off + r));
                P.target_tokens[i * (P.k_max + 1) + r] = tr;
                if (a < 0 && r < k && P.draft[i * P.k_max + r] != tr) a = r;
              }
              if (a < 0) a = k;
              P.accept_len[i] = a;
              if (P.commit) {
                int* s = P.seq + (size_t)slot * P.max_seq_len;
                int wpos = P.n_seq[slot];
                for (int r = 0; r < a && wpos < P.max_seq_len; ++r) s[wpos++] = P.draft[i * P.k_max + r];
                if (wpos < P.max_seq_len) s[wpos++] = argmax_key_index(__ldcg(P.keys + off + a));
                P.n_seq[slot] = wpos;
              }
            }
          } else if (et == 0 && P.mode != CALL_PREFILL) {
            P.draft_out[P.draft_step] = argmax_key_index(__ldcg(P.keys + P.logit_first_row));
          }
        }
      } else {
        // ---------------------------------------------------------------- GEMM epilogue
        empty_pending();
        const int pset = gph & 1;
        const KRange kr = phase_range(p.n_tiles, p.upt, p.kblocks, RANGE_UNIT_KB / kps, cta, G, p.ge_max);
        const int kb_begin = kr.begin, kb_end = kr.end;
        const int Ge = kr.ge;
        gemm_worked = kb_begin < kb_end;
        const int Tvalid = P.T;
        float* out_f32 = (p.epi == TC_LMHEAD) ? P.logits : reinterpret_cast<float*>(p.out);
        bf16* out_act = reinterpret_cast<bf16*>(p.out);
        unsigned long long* keys = P.keys;
        if (p.norm_in && kb_begin < kb_end) {
          // row statistics of the operand: merge the per-tile entries (published by the phase
          // that produced x) into mean and 1/std per row
          if (et == 0) ctl->bcast = W.wait_grid(bar_count, P.bar_base + (unsigned long long)ph * G) ? 1 : 0;
          epi_bar_sync();
          ok = ctl->bcast != 0;
          epi_bar_sync();
          if (!ok) break;
          // One warp per row, four rows per warp at a time.  A lane holds the tile entries lane and
          // lane + 32 of each row (all loads of the four rows in flight together; at most 64 tiles,
          // d <= 8192).  The merged mean is the count-weighted mean of the tiles' means, and the
          // merged M2 the sum of the tiles' M2 plus count * (tile mean - mean)^2: two warp sums
          // of non-negative or well-scaled terms, identical on every lane.
          for (int tb = quad; tb < Tvalid; tb += 16) {
            float4 sv[4][2];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              const int t = tb + 4 * r;
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const int tl = lane + 32 * e;
                sv[r][e] = (t < Tvalid && tl < P.stat_tiles) ? __ldcg(P.stats + (size_t)t * P.stat_tiles + tl) : make_float4(0.f, 0.f, 0.f, 0.f);
              }
            }
            float n[4], s1[4], m2[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              n[r] = sv[r][0].z + sv[r][1].z;
              s1[r] = sv[r][0].z * sv[r][0].x + sv[r][1].z * sv[r][1].x;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
              for (int r = 0; r < 4; ++r) { n[r] += __shfl_xor_sync(0xffffffffu, n[r], o); s1[r] += __shfl_xor_sync(0xffffffffu, s1[r], o); }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              s1[r] = s1[r] / fmaxf(n[r], 1.f);   // the row's mean
              const float d0 = sv[r][0].x - s1[r], d1 = sv[r][1].x - s1[r];
              m2[r] = (sv[r][0].y + sv[r][0].z * d0 * d0) + (sv[r][1].y + sv[r][1].z * d1 * d1);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
              for (int r = 0; r < 4; ++r) m2[r] += __shfl_xor_sync(0xffffffffu, m2[r], o);
            }
            if (lane == 0) {
#pragma unroll
              for (int r = 0; r < 4; ++r) {
                const int t = tb + 4 * r;
                if (t < Tvalid) {
                  if (P.norm_kind == 0) { ctl->mu[t] = s1[r]; ctl->rstd[t] = 1.0f / sqrtf(m2[r] / (float)P.d + P.eps); }
                  else { ctl->mu[t] = 0.f; ctl->rstd[t] = 1.0f / sqrtf((m2[r] + n[r] * s1[r] * s1[r]) / (float)P.d + P.eps); }
                }
              }
            }
          }
          epi_bar_sync();
        }
        if (tracing) tr[3] = globaltimer_ns();
        bool first_seg = true;
        int kb = kb_begin;
        const unsigned tot32 = (unsigned)(p.n_tiles * p.upt), ge32 = (unsigned)Ge;
        // first stage of CTA c's range (units * Ge < 2^32, checked on the host)
        auto rb = [&](unsigned c) { return (unsigned)unit_to_stage((tot32 * c) / ge32, p.upt, p.kblocks, RANGE_UNIT_KB / kps); };
        const int er = et >> 3, cg = et & 7;
        while (kb < kb_end && ok) {
          const int tile = kb / p.kblocks, kk0 = kb - tile * p.kblocks;
          const int tile_first = tile * p.kblocks, tile_end = tile_first + p.kblocks;
          const int seg_end = tile_end < kb_end ? tile_end : kb_end;
          // The CTA that owns a tile's first k-block finishes the tile; a CTA whose segment starts
          // inside a tile (always the first segment of its range, so at most one per phase) parks
          // the partial sums in its slot and raises its flag.  The finisher's segment is the
          // last thing its range holds, so it reaches the tile when the others are done or
          // nearly so, and it adds their partials to its own in k order - a fixed order: results
          // do not depend on timing.
          const bool finisher = kk0 == 0, whole = finisher && seg_end == tile_end;
          // first output column of the tile and how many of its columns exist (a tile never
          // straddles two sources)
          int n0, ncols, src_s = 0, src_col0 = 0;
          if (p.dual) { n0 = tile * 64; ncols = min(64, p.N - n0); }
          else {
            int local = tile, col0 = 0, col1 = p.n_src > 1 ? p.src_col[1] : p.N;
            if (p.n_src > 1 && local >= p.src_tiles[0]) {
              local -= p.src_tiles[0]; src_s = 1; col0 = p.src_col[1]; col1 = p.n_src > 2 ? p.src_col[2] : p.N;
              if (p.n_src > 2 && local >= p.src_tiles[1]) { local -= p.src_tiles[1]; src_s = 2; col0 = p.src_col[2]; col1 = p.N; }
            }
            src_col0 = col0;
            n0 = col0 + local * BM; ncols = min(BM, (col1 - col0) - local * BM);
          }
          // The epilogue runs in a per-row mapping: thread (er, cg) owns row er of a 16-row chunk
          // and the float4 column groups cg, cg + 8, cg + 16, cg + 24 of the tile (for a gate/up
          // tile: two gate groups and the matching two up groups) - compact code with vector
          // accesses.  What it needs from memory (per-column constants, the old residual values
          // of the first chunk) is fetched here, before the accumulator is waited for, so that
          // the round trips overlap the MMAs instead of extending the chain that ends the phase.
          // (Nobody else writes this tile's columns of the residual during the phase.)
          float4 xq[4];
          const bool have_pre = p.epi == TC_ADD_F32;
          // QKV projection: cache row of this thread's row (k and v tiles) and the rotation
          // table entries of its column groups (q and k tiles), for the first chunk
          int kv_row0 = 0;
          float4 rc0a, rc0b, rs0a, rs0b;
          auto kv_row_of = [&](int t) { return cache_row_of(P, t); };
          auto rope_of = [&](int t, float4& c0, float4& s0, float4& c1, float4& s1) {
            // hd = 128: groups (0, 2) and (1, 3) pair up, at table columns cg*4 and 32 + cg*4;
            // hd = 64: groups (0, 1) and (2, 3), both at table column cg*4
            const int hh = P.hd / 2;
            const int i1 = P.hd == 128 ? 32 + cg * 4 : cg * 4;
            c0 = __ldcg(reinterpret_cast<const float4*>(P.rope_cs + (size_t)t * hh + cg * 4));
            s0 = __ldcg(reinterpret_cast<const float4*>(P.rope_sn + (size_t)t * hh + cg * 4));
            c1 = __ldcg(reinterpret_cast<const float4*>(P.rope_cs + (size_t)t * hh + i1));
            s1 = __ldcg(reinterpret_cast<const float4*>(P.rope_sn + (size_t)t * hh + i1));
          };
          if (finisher && p.qkv_prep && er < Tvalid) {
            if (src_s >= 1) kv_row0 = kv_row_of(er);
            if (P.rope && src_s < 2) rope_of(er, rc0a, rs0a, rc0b, rs0b);
          }
          if (finisher) {
            const int mc = p.dual ? (m & 63) : m;
            const bool m_on = mc < ncols;
            if (p.norm_in) {
              const int ncol = (p.dual && m >= 64) ? p.N + n0 + mc : n0 + mc;
              ctl->utile[m] = (p.u && m_on) ? p.u[ncol] : 0.f;
              ctl->ctile[m] = (p.c && m_on) ? p.c[ncol] : 0.f;
            }
            if (have_pre) {
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const int col = (cg + 8 * q) * 4;
                xq[q] = (er < Tvalid && col < ncols) ? __ldcg(reinterpret_cast<const float4*>(out_f32 + (size_t)er * p.ldo + n0 + col))
                                                     : make_float4(0.f, 0.f, 0.f, 0.f);
              }
              ctl->gtile[m] = (p.next_g && m_on) ? p.next_g[n0 + mc] : 0.f;
            }
          }
          W.wait(ctl->acc_full + buf, (acc_bits >> buf) & 1u);
          __syncwarp();   // lanes may leave the wait an iteration apart; the barriers below want whole warps
          ok = group_ok(ctl, et);   // (its barriers also publish the staged constants)
          if (!ok) break;
          if (tracing && first_seg) { tr[4] = globaltimer_ns(); first_seg = false; }
          acc_bits ^= 1u << buf;
          tc_fence_after();
          const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * 2 * P.t_box);
          unsigned long long* tra = (MK_TRACE_PTR(P.trace) && et == 0 && !whole) ? MK_TRACE_PTR(P.trace) + (size_t)2 * P.n_phases * 8 + ((size_t)cta * P.n_phases + ph) * 8 : nullptr;
          if (!finisher) {
            if (tra) tra[4] = globaltimer_ns();
            float* mine = slot_of(pset, (unsigned)cta);
            for (int c0 = 0; c0 < Tvalid; c0 += 16) {   // only rows that exist
              float v[16];
              tmem_ld16(taddr + (uint32_t)c0, v);
              {
                float vl[16];
                tmem_ld16(taddr + (uint32_t)(P.t_box + c0), vl);
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] += vl[j];
              }
              const int jn = min(16, Tvalid - c0);
#pragma unroll
              for (int j = 0; j < 16; ++j) if (j < jn) st_relaxed_f32(mine + (size_t)(c0 + j) * BM + m, v[j]);
            }
            // (no flag and no fence: the finisher polls the values themselves)
            tc_fence_before();
            if (lane == 0) mbar_arrive(ctl->acc_empty + buf);
            if (tra) tra[5] = globaltimer_ns();
          } else {
            unsigned last_c = (unsigned)cta;   // CTAs cta + 1 .. last_c hold the tile's other segments
            if (!whole) while (last_c + 1 < ge32 && rb(last_c + 1) < (unsigned)tile_end) ++last_c;
            if (!whole) { pend_first = (unsigned)cta + 1u; pend_last = last_c; pend_set = pset; }   // (at most one split tile is finished per phase)
            for (int c0 = 0; c0 < Tvalid; c0 += 16) {
              {
                float v[16];
                tmem_ld16(taddr + (uint32_t)c0, v);
                {
                  float vl[16];
                  tmem_ld16(taddr + (uint32_t)(P.t_box + c0), vl);
#pragma unroll
                  for (int j = 0; j < 16; ++j) v[j] += vl[j];
                }
                if (c0 + 16 >= Tvalid) {   // accumulator drained: the MMA warp may reuse it
                  tc_fence_before();
                  if (lane == 0) mbar_arrive(ctl->acc_empty + buf);
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) vt[j * VT_LD + m] = v[j];
              }
              epi_bar_sync();   // the exchange tile is complete
              if (tra && !whole && c0 == 0) tra[1] = globaltimer_ns();
              {
                // Each phase runs this code once per tile, so its instruction fetch is what it costs:
                // the loads that must be in flight together are unrolled, everything per column group
                // is a rolled loop over the four groups of the thread (the sums wait in the exchange tile).
                const int t = c0 + er;
                const bool row_on = t < Tvalid;
                float* vrow = vt + er * VT_LD;
                const bool add_res = p.epi == TC_ADD_F32;
                if (!whole || add_res) {
                  float4 a[4];
                  bool on[4];
#pragma unroll
                  for (int q = 0; q < 4; ++q) {
                    const int col = (cg + 8 * q) * 4;
                    on[q] = row_on && (p.dual ? (col & 63) < ncols : col < ncols);
                    a[q] = on[q] ? *reinterpret_cast<const float4*>(vrow + col) : make_float4(0.f, 0.f, 0.f, 0.f);
                  }
                  if (!whole) {
                    // The other segments' partial sums, six segments' loads in flight together, added in k
                    // order.  A slot element reads PARTIAL_EMPTY until its producer has stored the sum: when
                    // one does, the thread waits on a single element (little traffic while others still
                    // stream weights) and then looks at all of them again.  All waits are bounded.
                    for (unsigned c = (unsigned)cta + 1; c <= last_c; c += 6) {
                      uint4 tmp[6][4];
                      const float* probe = slot_of(pset, min(c + 5, last_c)) + (size_t)(row_on ? t : 0) * BM + cg * 4;
                      long long t0 = 0;
                      bool timing = false, give_up = false;
                      while (true) {
                        uint32_t mx = 0u;
#pragma unroll
                        for (int u = 0; u < 6; ++u) {
                          const float* part = slot_of(pset, min(c + u, last_c)) + (size_t)(row_on ? t : 0) * BM;
#pragma unroll
                          for (int q = 0; q < 4; ++q) {
                            tmp[u][q] = (on[q] && c + u <= last_c) ? ld_relaxed_u4(part + (cg + 8 * q) * 4) : make_uint4(0u, 0u, 0u, 0u);
                            mx = max(max(mx, max(tmp[u][q].x, tmp[u][q].y)), max(tmp[u][q].z, tmp[u][q].w));
                          }
                        }
                        if (mx != PARTIAL_EMPTY || give_up) break;
                        do {
                          if (!timing) { t0 = clock64(); timing = true; }
                          if (W.poll_abort(t0)) { W.note(3u, (unsigned)ph, (unsigned)cta, last_c, (unsigned)tile); give_up = true; break; }   // (the verdict follows the chunk's last barrier)
                          __nanosleep(32);
                        } while (ld_relaxed_u4(probe).x == PARTIAL_EMPTY);
                      }
#pragma unroll
                      for (int u = 0; u < 6; ++u) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                          a[q].x += __uint_as_float(tmp[u][q].x); a[q].y += __uint_as_float(tmp[u][q].y);
                          a[q].z += __uint_as_float(tmp[u][q].z); a[q].w += __uint_as_float(tmp[u][q].w);
                        }
                      }
                    }
                    if (tra && c0 == 0) tra[2] = globaltimer_ns();
                  }
                  if (tra) {
                    asm volatile("" ::"f"(a[0].x), "f"(a[0].w), "f"(a[1].x), "f"(a[1].w), "f"(a[2].x), "f"(a[2].w), "f"(a[3].x), "f"(a[3].w));
                    tra[6] = globaltimer_ns();
                  }
                  if (add_res) {
                    // residual update (a residual GEMM has no folded normalisation)
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                      if (on[q]) {
                        const size_t o = (size_t)t * p.ldo + n0 + (cg + 8 * q) * 4;
                        const float4 x4 = xq[q];   // (requested before the accumulator was waited for, or during the previous chunk)
                        a[q] = make_float4(x4.x + a[q].x, x4.y + a[q].y, x4.z + a[q].z, x4.w + a[q].w);
                        *reinterpret_cast<float4*>(out_f32 + o) = a[q];
                      }
                    }
                  }
#pragma unroll
                  for (int q = 0; q < 4; ++q)
                    if (on[q]) *reinterpret_cast<float4*>(vrow + (cg + 8 * q) * 4) = a[q];   // (this thread's own slots)
                  if (add_res && c0 + 16 < Tvalid) {
                    // calls of more than 16 rows: the next chunk's old residual values are requested now,
                    // so that they do not add an L2 round trip to that chunk
                    const int tn = t + 16;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                      const int col = (cg + 8 * q) * 4;
                      xq[q] = (tn < Tvalid && col < ncols) ? __ldcg(reinterpret_cast<const float4*>(out_f32 + (size_t)tn * p.ldo + n0 + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                  }
                }
                // column group `col` of this thread's row, with the folded normalisation
                // y = rstd_t * (acc - mean_t * u[n]) + c[n] where the GEMM has one
                const float rs = (p.norm_in && row_on) ? ctl->rstd[t] : 1.0f, mu = (p.norm_in && row_on) ? ctl->mu[t] : 0.f;
                auto group = [&](int col) -> float4 {
                  float4 v = *reinterpret_cast<const float4*>(vrow + col);
                  if (p.norm_in) {
                    const float4 u4 = *reinterpret_cast<const float4*>(ctl->utile + col);
                    const float4 c4 = *reinterpret_cast<const float4*>(ctl->ctile + col);
                    v.x = rs * (v.x - mu * u4.x) + c4.x; v.y = rs * (v.y - mu * u4.y) + c4.y;
                    v.z = rs * (v.z - mu * u4.z) + c4.z; v.w = rs * (v.w - mu * u4.w) + c4.w;
                  }
                  return v;
                };
                if (add_res) {
                  // with a following normalised GEMM: its operand bf16(x * gain) and this tile's row
                  // statistics (count, mean, centred sum of squares; two passes over the row's 128 values)
                  if (p.next_g) {
                    float cnt = 0.f, sum = 0.f;
#pragma unroll 1
                    for (int q = 0; q < 4; ++q) {
                      const int col = (cg + 8 * q) * 4;
                      if (row_on && col < ncols) {
                        const float4 x4 = *reinterpret_cast<const float4*>(vrow + col);
                        const float4 g4 = *reinterpret_cast<const float4*>(ctl->gtile + col);
                        store_split4(P.h, (size_t)t * p.ldo + n0 + col, (size_t)P.lo_row * p.ldo, make_float4(x4.x * g4.x, x4.y * g4.y, x4.z * g4.z, x4.w * g4.w));
                        cnt += 4.f; sum += (x4.x + x4.y) + (x4.z + x4.w);
                      }
                    }
                    if (tra) { asm volatile("" ::"f"(sum), "f"(cnt)); tra[7] = globaltimer_ns(); }
#pragma unroll
                    for (int o = 1; o < 8; o <<= 1) { cnt += __shfl_xor_sync(0xffffffffu, cnt, o); sum += __shfl_xor_sync(0xffffffffu, sum, o); }
                    const float mean = cnt > 0.f ? sum / cnt : 0.f;
                    float m2 = 0.f;
#pragma unroll 1
                    for (int q = 0; q < 4; ++q) {
                      const int col = (cg + 8 * q) * 4;
                      if (row_on && col < ncols) {
                        const float4 x4 = *reinterpret_cast<const float4*>(vrow + col);
                        const float d0 = x4.x - mean, d1 = x4.y - mean, d2 = x4.z - mean, d3 = x4.w - mean;
                        m2 += (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
                      }
                    }
#pragma unroll
                    for (int o = 1; o < 8; o <<= 1) m2 += __shfl_xor_sync(0xffffffffu, m2, o);
                    if (cg == 0 && row_on) P.stats[(size_t)t * P.stat_tiles + tile] = make_float4(mean, m2, cnt, 0.f);
                  }
                } else if (p.epi == TC_SWIGLU) {
                  // gate columns (cg + 8 q) * 4 of the tile's first half, the matching up columns 64 further
#pragma unroll 1
                  for (int q = 0; q < 2; ++q) {
                    const int col = (cg + 8 * q) * 4;
                    if (row_on && col < ncols) {
                      const float4 g4 = group(col), u4 = group(col + 64);
                      store_split4(out_act, (size_t)t * p.ldo + n0 + col, (size_t)P.lo_row * p.ldo,
                                   make_float4(silu_f(g4.x) * u4.x, silu_f(g4.y) * u4.y, silu_f(g4.z) * u4.z, silu_f(g4.w) * u4.w));
                    }
                  }
                } else if (p.epi == TC_LMHEAD) {
                  // logits (optional) and the row's running argmax; the vocabulary need not be a
                  // multiple of 4, so validity and stores are per element
                  unsigned long long key = 0ull;
#pragma unroll 1
                  for (int q = 0; q < 4; ++q) {
                    const int col = (cg + 8 * q) * 4;
                    const float4 v4 = group(col);
                    const float e4[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                      if (row_on && col + e < ncols) {
                        if (out_f32) out_f32[(size_t)t * p.ldo + n0 + col + e] = e4[e];
                        const unsigned long long k2 = argmax_key(e4[e], (uint32_t)(n0 + col + e));
                        key = k2 > key ? k2 : key;
                      }
                    }
                  }
#pragma unroll
                  for (int o = 1; o < 8; o <<= 1) {
                    const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
                    key = other > key ? other : key;
                  }
                  if (cg == 0 && key) atomicMax(keys + t, key);
                } else if (p.qkv_prep) {
                  // q: rotate, scale by 1/sqrt(hd), fp16, to the query buffer; k: rotate, fp16, to
                  // its row of the cache; v: fp16 to the cache.  The rotation pairs column i with
                  // i + hd/2 of a head; with hd = 128 (a tile is one head: groups 0 and 2, 1 and 3) or
                  // 64 (two heads: groups 0 and 1, 2 and 3) both columns of a pair belong to the same thread.
                  int kv_row = kv_row0;
                  float4 rca = rc0a, rcb = rc0b, rsa = rs0a, rsb = rs0b;
                  if (c0 != 0 && row_on) {
                    if (src_s >= 1) kv_row = kv_row_of(t);
                    if (P.rope && src_s < 2) rope_of(t, rca, rsa, rcb, rsb);
                  }
                  const float qscale = src_s == 0 ? 1.4426950408889634f / sqrtf((float)P.hd) : 1.0f;   // log2(e) / sqrt(hd): the softmax works in base 2
                  const int nq_all = P.Hq * P.hd, nkv_all = P.Hkv * P.hd;
                  __half* dst = (src_s == 0 ? P.q16 + (size_t)t * nq_all
                                            : reinterpret_cast<__half*>(src_s == 1 ? p.kc : p.vc) + (size_t)kv_row * nkv_all) + (n0 - src_col0);
#pragma unroll 1
                  for (int pi = 0; pi < 2; ++pi) {
                    const int col_lo = (P.hd == 128 ? cg + 8 * pi : cg + 16 * pi) * 4, col_hi = col_lo + (P.hd == 128 ? 64 : 32);
                    float4 lo = group(col_lo), hi = group(col_hi);
                    if (P.rope && src_s < 2) {
                      const float4 cs = pi ? rcb : rca, sn = pi ? rsb : rsa;
                      const float4 l = lo, h = hi;
                      lo = make_float4(l.x * cs.x - h.x * sn.x, l.y * cs.y - h.y * sn.y, l.z * cs.z - h.z * sn.z, l.w * cs.w - h.w * sn.w);
                      hi = make_float4(h.x * cs.x + l.x * sn.x, h.y * cs.y + l.y * sn.y, h.z * cs.z + l.z * sn.z, h.w * cs.w + l.w * sn.w);
                    }
                    if (row_on && col_lo < ncols)
                      *reinterpret_cast<uint2*>(dst + col_lo) = make_uint2(pack_f16x2(lo.x * qscale, lo.y * qscale), pack_f16x2(lo.z * qscale, lo.w * qscale));
                    if (row_on && col_hi < ncols)
                      *reinterpret_cast<uint2*>(dst + col_hi) = make_uint2(pack_f16x2(hi.x * qscale, hi.y * qscale), pack_f16x2(hi.z * qscale, hi.w * qscale));
                  }
                } else {
#pragma unroll 1
                  for (int q = 0; q < 4; ++q) {
                    const int col = (cg + 8 * q) * 4;
                    if (row_on && col < ncols) {
                      const float4 v4 = group(col);
                      const size_t o = (size_t)t * p.ldo + n0 + col;
                      if (p.epi == TC_STORE_F32) *reinterpret_cast<float4*>(out_f32 + o) = v4;
                      else store_split4(out_act, o, (size_t)P.lo_row * p.ldo, make_float4(gelu_erf(v4.x), gelu_erf(v4.y), gelu_erf(v4.z), gelu_erf(v4.w)));
                    }
                  }
                }
              }
              // one verdict for the 128 threads (a poll above may have run out in some of them; one that
              // thread 0 misses here is seen at the next verdict or at the end of the kernel)
              if (et == 0) ctl->bcast = ctl->abort_flag ? 0 : 1;
              epi_bar_sync();   // (the exchange tile is reused by the next chunk)
              ok = ctl->bcast != 0;
              if (!ok) break;
            }
            if (tra) tra[3] = globaltimer_ns();
          }
          if (!ok) break;
          buf ^= 1;
          kb = seg_end;
        }
      }
      if (!ok) break;
      if (tracing) tr[1] = globaltimer_ns();
      // every CTA's completion time of the phase, after the two detailed traces
      if (MK_TRACE_PTR(P.trace) && et == 0) MK_TRACE_PTR(P.trace)[(size_t)2 * P.n_phases * 8 + ((size_t)cta * P.n_phases + ph) * 8] = globaltimer_ns();
      // Publish this CTA's part of the phase.  A CTA may arrive for phase ph only once every
      // CTA has arrived for phase ph-1: otherwise CTAs without work in two consecutive GEMM
      // phases would run ahead and their arrivals would be mistaken for the slower CTAs' ones
      // (one monotonic counter serves all phases).  For a CTA that had GEMM work the wait is
      // already satisfied - its own activation tiles were gated on the same count.
      // The release below is cumulative: it covers the other compute threads' stores, which the
      // barrier orders before it.  A CTA that had GEMM work in this phase already knows that
      // barrier ph-1 completed (its activation tiles were loaded after that), so only idle CTAs
      // look at the counter.
#ifdef STAIRS_TRACE
      if (tracing && cta != 0) tr[5] = globaltimer_ns();
#endif
      fence_proxy_async();   // later TMA (async proxy) reads of these generic-proxy writes
#ifdef STAIRS_TRACE
      if (tracing && cta != 0) tr[6] = globaltimer_ns();
#endif
      if (et < PH_WORDS) ctl->phc[(ph + 1) & 1][et] = next_word;   // (the barriers below publish it)
      if (ph > 0 && p.kind == PH_GEMM && !gemm_worked) {
        if (et == 0) ctl->bcast = W.wait_grid(bar_count, P.bar_base + (unsigned long long)ph * G) ? 1 : 0;
        epi_bar_sync();
        ok = ctl->bcast != 0;
        epi_bar_sync();
        if (!ok) break;
      } else {
        epi_bar_sync();
      }
#ifdef STAIRS_TRACE
      if (tracing && cta != 0) tr[7] = globaltimer_ns();
#endif
      if (et == 0) red_release_add_u64(P.bar, 1ull);
      if (tracing) tr[2] = globaltimer_ns();
      waited = false;
      if (p.kind == PH_GEMM) ++gph;
    }
    if (ok) { empty_pending(); if (aph > 0) empty_own_states((aph - 1) & 1); }   // (after an abort the host empties every slot)
  }

  // ================================================================== teardown
  tc_fence_before();
  __syncthreads();
  if (ctl->abort_flag) {
    if (threadIdx.x == 0) {
      atomicExch(P.bar + 1, 1ull);   // tell the other CTAs
      // STAIRS_ETIMEOUT, or STAIRS_ENOSPC when the first note is the attention-scratch guard's
      *reinterpret_cast<volatile unsigned int*>(P.status + STATUS_ERROR) =
          *reinterpret_cast<volatile unsigned int*>(P.status + STATUS_WHERE) == 4u ? 2u : 5u;
      __threadfence_system();
      // let the copies in flight land before the CTA's shared memory is given up (a stage whose
      // activation tile was never issued cannot complete: the loop is bounded, by at least ~1 ms so
      // that a very short wait limit still leaves the copies time to finish)
      const long long t0 = clock64();
      const unsigned long long drain_limit = P.wait_limit > 2000000ull ? P.wait_limit : 2000000ull;
      int s = p_stage; uint32_t phs = p_phase;
      for (int i = 0; i < stages && i < issued; ++i) {
        if (--s < 0) { s = stages - 1; phs ^= 1; }
        while (!mbar_try(ctl->full + s, phs)) {
          if ((unsigned long long)(clock64() - t0) > drain_limit) break;
        }
      }
    }
    __syncthreads();
  }
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, tmem_cols); }
}

inline size_t smem_bytes(int t_box, int stages, int hd, int dbl, int kps, int tma = 0, int nbuf = 0, int tc_q_rows = 0) {
  return 1024 + (size_t)stages * kps * (A_STAGE_BYTES + (size_t)2 * t_box * BK * 2) + MK_XCH_BYTES + ((sizeof(Ctl) + 127) & ~(size_t)127) +
         AttnSmem::bytes(hd, dbl, tma, nbuf, tc_q_rows) + 64;
}
inline int pick_stages(int t_box, int hd, int dbl, int kps, int tma = 0, int nbuf = 0, int tc_q_rows = 0) {
  int s = MAX_STAGES;
  while (s > 1 && smem_bytes(t_box, s, hd, dbl, kps, tma, nbuf, tc_q_rows) > (size_t)SMEM_LIMIT) --s;
  return s;
}
// k-blocks per stage: two while at least three stages still fit (small row boxes), else one
inline int pick_kps(int t_box, int hd, int dbl) { return pick_stages(t_box, hd, dbl, 2) >= 3 ? 2 : 1; }

}  // namespace mk
}  // namespace stairs
