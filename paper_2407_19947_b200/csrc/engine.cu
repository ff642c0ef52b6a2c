// Host engine and C-ABI of the stairs library: context, workspace layout, KV page
// allocator, the per-pass kernel sequence, draft / validate / generate.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <new>
#include <string>
#include <tuple>
#include <type_traits>
#include <vector>

#include "../../include/stairs.h"
#include "../../include/stairs_debug.h"
#include "common.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "kernels_basic.cuh"
#include "megakernel.cuh"

using namespace stairs;

namespace {

thread_local std::string g_init_error;

struct LayerMaps { CUtensorMap wq, wk, wv, wo, w1, w3, w2; };

constexpr int TC_GRID_MAX = 160;        // scratch is sized for at most this many CTAs
constexpr int TC_COUNTERS = 1 << 16;    // tiles per GEMM the split bookkeeping can hold

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int MK_MAX_ROWS = 64;          // rows per call the persistent kernel handles
constexpr int MK_TBOX_SLOTS = MK_MAX_ROWS / 16;
constexpr int MK_PROG_SLOTS = MK_TBOX_SLOTS * 2;   // one program per (row box, k-blocks per stage)

struct DevModel {
  float* rope_inv = nullptr;     // device: theta^(-2i/hd), i < hd/2
  float* ln_aux = nullptr;       // device: LayerNorm u/c vectors (see build_program)
  bf16* w13 = nullptr;           // device: SwiGLU models, per layer [tiles][64 gate rows | 64 up rows][d] (see k_pack_gate_up)
  size_t w13_layer = 0;          // elements per layer
  std::vector<const bf16*> w13_ptr;   // per layer: its packed matrix (possibly another model's, for shared layers)
  bool prog_built[MK_PROG_SLOTS] = {};
  char* prog_base = nullptr;     // device: per t_box slot, phases followed by tensor maps
  size_t prog_slot_bytes = 0, prog_maps_off = 0;
  int n_phases = 0;
  std::vector<LayerMaps> maps;   // tensor maps of the bf16 weight matrices (tensor-core path)
  CUtensorMap head_map{};
  stairs_model m{};
  bool present = false;
  stairs_weights w{};
  std::vector<stairs_layer_w> layers;
  char* kpool = nullptr;  // [n_layers][pool_tokens][Hkv*hd] elements of the weight dtype
  char* vpool = nullptr;
  size_t kv_layer_bytes = 0;
};

struct Layout {
  size_t status, seq, n_seq, page_table, tok, pos, req, val_req, val_k, val_off, keys, x, h, qkv, q,
      o, ff, logits, draft_buf, tt_buf, al_buf, gemm_partial, gemm_counters, mk_partial, mk_partial_bytes, mk_bar, attn_part, prog_t, prog_d, mk_trace, mk_stats, rope_t, rope_d, aux_t, aux_d, w13_t, w13_d, kv_t_k, kv_t_v, kv_d_k, kv_d_v, total;
  int max_rows, logit_rows, max_pages, n_pages, t_box_max, attn_units, stat_tiles;
  size_t prog_slot_t, prog_slot_d, prog_maps_off_t, prog_maps_off_d;
  size_t kv_t_layer, kv_d_layer;
  size_t attn_part_bytes;
};

}  // namespace

struct stairs_ctx {
  stairs_config cfg{};
  DevModel target, draft;
  Layout lay{};
  cudaStream_t stream = nullptr;
  char* ws = nullptr;
  std::string err;
  int64_t launches = 0;
  // host mirrors
  std::vector<int> free_pages;
  std::vector<std::vector<int>> pages;  // per slot
  std::vector<int> n_seq_ub;            // upper bound of the device-side sequence length
  std::vector<char> active;
  // profiling
  bool profile = false;
  std::vector<cudaEvent_t> ev;
  int ev_used = 0;
  cudaEvent_t call_begin = nullptr, call_end = nullptr;
  bool in_validate = false;
  // tensor-core path
  bool use_tc = false;
  int sm_count = 0;
  EncodeTiledFn encode = nullptr;
  std::map<std::tuple<const void*, int, int>, CUtensorMap> act_maps;
  unsigned int* status_host = nullptr;  // pinned, device-visible status words
  unsigned int* status_dev = nullptr;
  // pinned, device-visible block of the host-buffer entry points: drafts in (staged for one
  // asynchronous copy), target tokens and accept lengths out (written by the kernel itself)
  int* io_host = nullptr;
  int* io_dev = nullptr;
  size_t io_draft = 0, io_tt = 0, io_al = 0;   // offsets in ints
  unsigned long long wait_limit = 0;
  bool use_mk = false;
  bool draft_shares_kv = false;      // early-exit assistant on the persistent kernel: it uses the main model's K/V pools
  unsigned long long bar_base = 0;   // grid-barrier arrivals consumed by earlier launches
  int kps_force = 0;                 // tuning: k-blocks per pipeline stage (0 = chosen per row box)
  int att_nbuf_force = 0;            // tuning: K/V chunk buffers of the attention phases (0 = chosen from the context length)
  int att_tc_force = 0;              // tuning: 1 = tcgen05 attention for every call it can serve
  int att_tc_off = 0;                // tuning: 1 = attention contractions on mma.sync even where the tcgen05 path applies
  int att_tma_off = 0;               // tuning: 1 = stage K/V with 16-byte copies from the compute warps even where bulk copies apply
};

namespace {

int fail(stairs_ctx* c, int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (c) c->err = buf; else g_init_error = buf;
  return code;
}

#define CK(call)                                                                              \
  do {                                                                                        \
    cudaError_t e_ = (call);                                                                  \
    if (e_ != cudaSuccess)                                                                    \
      return fail(ctx, STAIRS_ECUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_),  \
                  __FILE__, __LINE__);                                                        \
  } while (0)

size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }
int esize(const stairs_model& m) { return m.wdtype == 0 ? 4 : 2; }

const char* check_model(const stairs_model& m) {
  if (m.n_layers < 0 || m.d_model <= 0 || m.n_heads <= 0 || m.n_kv_heads <= 0 || m.head_dim <= 0 ||
      m.d_ff <= 0 || m.vocab <= 0)
    return "model dimensions must be positive";
  if (m.n_heads % m.n_kv_heads) return "n_heads must be a multiple of n_kv_heads";
  if (m.head_dim % 8 || m.head_dim > 256) return "head_dim must be a multiple of 8 and <= 256";
  if (m.d_model % 8 || m.d_ff % 8) return "d_model and d_ff must be multiples of 8";
  if (m.norm < 0 || m.norm > 1 || m.act < 0 || m.act > 1 || m.pos < 0 || m.pos > 1) return "norm/act/pos out of range";
  if (m.wdtype < 0 || m.wdtype > 1) return "wdtype must be 0 (fp32) or 1 (bf16)";
  if (m.pos == 0 && m.max_pos <= 0) return "max_pos must be positive with learned positions";
  return nullptr;
}

// Upper bound of the attention units of one request with `rows` rows in the persistent kernel: the
// kernel picks chunks per unit so that kv heads x position ranges fit the grid (or, for contexts
// too long for that, at most twice the grid: stairs_init checks this); the rows of the call can
// add one more range per kv head.
int attn_unit_bound(int hkv, int gq, int rows, int qblk = mk::ATT_QBLK) {
  const int n_qblk = (rows * gq + qblk - 1) / qblk;
  return (2 * TC_GRID_MAX + 2 * hkv) * std::max(n_qblk, 1);
}

bool compute_layout(const stairs_config& c, Layout* L, const char** why) {
  *why = nullptr;
  if (c.struct_size != sizeof(stairs_config)) { *why = "struct_size does not match this library"; return false; }
  if ((*why = check_model(c.target))) return false;
  const bool has_draft = c.draft.n_layers > 0;
  if (has_draft) {
    if ((*why = check_model(c.draft))) return false;
    if (c.draft.d_model != c.target.d_model || c.draft.vocab != c.target.vocab ||
        c.draft.wdtype != c.target.wdtype || c.draft.norm != c.target.norm ||
        c.draft.act != c.target.act || c.draft.pos != c.target.pos) {
      *why = "draft must share d_model, vocab, wdtype and the norm/act/pos family with the target";
      return false;
    }
  }
  if (c.max_requests <= 0 || c.max_seq_len < 4 || c.k_max < 0 || c.k_max > 63) {
    *why = "max_requests > 0, max_seq_len >= 4 and 0 <= k_max <= 63 required"; return false;
  }
  const int pt = c.kv_page_tokens;
  if (pt != 16 && pt != 32 && pt != 64 && pt != 128) { *why = "kv_page_tokens must be 16, 32, 64 or 128"; return false; }
  if (c.target.pos == 0 && c.max_seq_len > c.target.max_pos) { *why = "max_seq_len exceeds max_pos of the learned positions"; return false; }
  if (c.kv_pages < 0 || c.prefill_chunk < 0) { *why = "kv_pages and prefill_chunk must not be negative"; return false; }
  const int chunk = c.prefill_chunk > 0 ? c.prefill_chunk : 256;
  L->max_rows = (std::max(std::max(chunk, c.max_requests * (c.k_max + 1)), 2) + 15) / 16 * 16;
  if (c.target.wdtype == 1) L->max_rows = std::max(L->max_rows, MK_MAX_ROWS);   // prefill passes of the persistent kernel
  L->t_box_max = std::min(256, L->max_rows);
  L->logit_rows = std::max(c.max_requests * (c.k_max + 1), 1);
  L->max_pages = (c.max_seq_len + pt - 1) / pt;
  L->n_pages = c.kv_pages > 0 ? c.kv_pages : L->max_pages * c.max_requests;
  const stairs_model& t = c.target;
  const stairs_model& d = c.draft;
  auto mx = [&](int a, int b) { return has_draft ? std::max(a, b) : a; };
  const size_t es = esize(t);
  const size_t dm = t.d_model;
  const size_t nq = mx(t.n_heads * t.head_dim, d.n_heads * d.head_dim);
  const size_t nqkv = mx((t.n_heads + 2 * t.n_kv_heads) * t.head_dim, (d.n_heads + 2 * d.n_kv_heads) * d.head_dim);
  const size_t ff = mx(t.d_ff, d.d_ff);
  const size_t R = L->max_rows;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  L->status = take(STATUS_WORDS * 4);
  L->mk_bar = take(64);
  L->seq = take((size_t)c.max_requests * c.max_seq_len * 4);
  L->n_seq = take((size_t)c.max_requests * 4);
  L->page_table = take((size_t)c.max_requests * L->max_pages * 4);
  L->tok = take(R * 4); L->pos = take(R * 4); L->req = take(R * 4);
  L->val_req = take((size_t)c.max_requests * 4);
  L->val_k = take((size_t)c.max_requests * 4);
  L->val_off = take((size_t)c.max_requests * 4);
  L->keys = take(R * 8);
  L->x = take(R * dm * 4);
  const size_t parts = t.wdtype == 1 ? 2 : 1;   // bf16 GEMM operands are stored as hi + lo parts
  L->h = take(parts * R * dm * es);
  L->qkv = take(R * nqkv * 4);
  L->q = take(R * nq * es);
  L->o = take(parts * R * nq * es);
  L->ff = take(parts * R * ff * es);
  L->logits = take((size_t)L->logit_rows * t.vocab * 4);
  L->draft_buf = take((size_t)c.max_requests * std::max(c.k_max, 1) * 4);
  L->tt_buf = take((size_t)c.max_requests * (c.k_max + 1) * 4);
  L->al_buf = take((size_t)c.max_requests * 4);
  L->gemm_partial = take(t.wdtype == 1 ? (size_t)TC_GRID_MAX * 2 * L->t_box_max * tc::BM * 4 : 0);
  L->gemm_counters = take(t.wdtype == 1 ? (size_t)TC_COUNTERS * 4 : 0);
  // split-tile partial sums of the persistent kernel: two sets (alternate GEMM phases) of one slot per CTA;
  // every element holds the "empty" pattern between uses
  L->mk_partial_bytes = t.wdtype == 1 ? (size_t)2 * TC_GRID_MAX * L->t_box_max * tc::BM * 4 : 0;
  L->mk_partial = take(L->mk_partial_bytes);
  {
    // persistent-kernel scratch: attention unit states and the per-(model, row box) programs
    const int hkv = mx(t.n_kv_heads, d.n_kv_heads), hdm = mx(t.head_dim, d.head_dim);
    const int gq = mx(t.n_heads / t.n_kv_heads, has_draft ? d.n_heads / d.n_kv_heads : 1);
    // A request with R rows has at most (2 * grid + 2 * Hkv) * ceil(R * G / query block) units (see
    // attn_unit_bound).  A validate call holds up to max_requests requests of k_max + 1 rows; a
    // prefill pass of the persistent kernel is one request of MK_MAX_ROWS rows.
    const int rows_req = std::min(c.k_max + 1, MK_MAX_ROWS);
    L->attn_units = std::max(c.max_requests * attn_unit_bound(hkv, gq, rows_req), attn_unit_bound(hkv, gq, MK_MAX_ROWS));
    // (the tcgen05 attention path has fewer units of 128 query rows each: sized for whichever is larger)
    const int units_tc = std::max(c.max_requests * attn_unit_bound(hkv, gq, rows_req, mk::ATT_QBLK_TC), attn_unit_bound(hkv, gq, MK_MAX_ROWS, mk::ATT_QBLK_TC));
    L->attn_part_bytes = std::max((size_t)L->attn_units * mk::ATT_QBLK, (size_t)units_tc * mk::ATT_QBLK_TC) * (hdm + 4) * 4;
    L->attn_part = take(t.wdtype == 1 ? 2 * L->attn_part_bytes : 0);   // two sets (alternate attention phases), every word "empty" between uses
    auto prog = [&](const stairs_model& m, size_t* maps_off) {
      const size_t ph = align_up((size_t)(8 * std::max(m.n_layers, 1) + 4) * sizeof(mk::Phase), 128);
      *maps_off = ph;
      return ph + (size_t)(9 * std::max(m.n_layers, 1) + 4) * sizeof(CUtensorMap);   // 7 weight and 2 K/V pool maps per layer
    };
    L->prog_slot_t = t.wdtype == 1 ? prog(t, &L->prog_maps_off_t) : 0;
    L->prog_slot_d = (t.wdtype == 1 && has_draft) ? prog(d, &L->prog_maps_off_d) : 0;
    L->prog_t = take(L->prog_slot_t * MK_PROG_SLOTS);
    L->prog_d = take(L->prog_slot_d * MK_PROG_SLOTS);
    L->mk_trace = take(t.wdtype == 1 ? (size_t)(2 * 8 + 8 * TC_GRID_MAX) * (8 * std::max(t.n_layers, 1) + 4) * 8 : 0);
    L->stat_tiles = (t.d_model + tc::BM - 1) / tc::BM;
    L->mk_stats = take(t.wdtype == 1 ? (size_t)MK_MAX_ROWS * L->stat_tiles * 16 : 0);
    L->rope_t = take(t.wdtype == 1 ? (size_t)t.head_dim * 2 * (1 + 2 * 64) : 0);   // inverse frequencies, then cos and sin of 64 rows
    L->rope_d = take((t.wdtype == 1 && has_draft) ? (size_t)d.head_dim * 2 * (1 + 2 * 64) : 0);
    // LayerNorm models: u = W.gain and c = W.bias per normalised GEMM (fp32)
    auto aux = [&](const stairs_model& m) {
      if (m.norm != 0) return (size_t)0;
      const size_t nqkv2 = (size_t)(m.n_heads + 2 * m.n_kv_heads) * m.head_dim, f2 = (size_t)m.d_ff * (m.act == 1 ? 2 : 1);
      return ((nqkv2 + f2) * m.n_layers + m.vocab) * 2 * 4;
    };
    L->aux_t = take(t.wdtype == 1 ? aux(t) : 0);
    L->aux_d = take((t.wdtype == 1 && has_draft) ? aux(d) : 0);
    // SwiGLU models: gate and up rows interleaved per 64-row tile, so the persistent kernel streams
    // them as one matrix (a one-time repack of borrowed weights into the workspace)
    auto w13 = [&](const stairs_model& m) {
      return m.act == 1 ? (size_t)((m.d_ff + 63) / 64) * 128 * m.d_model * 2 * m.n_layers : (size_t)0;
    };
    L->w13_t = take(t.wdtype == 1 ? w13(t) : 0);
    L->w13_d = take((t.wdtype == 1 && has_draft) ? w13(d) : 0);
  }
  const size_t pool_tokens = (size_t)L->n_pages * pt;
  L->kv_t_layer = pool_tokens * t.n_kv_heads * t.head_dim * es;
  L->kv_t_k = take(L->kv_t_layer * t.n_layers);
  L->kv_t_v = take(L->kv_t_layer * t.n_layers);
  L->kv_d_layer = has_draft ? pool_tokens * d.n_kv_heads * d.head_dim * es : 0;
  L->kv_d_k = take(L->kv_d_layer * (has_draft ? d.n_layers : 0));
  L->kv_d_v = take(L->kv_d_layer * (has_draft ? d.n_layers : 0));
  L->total = off;
  return true;
}

// ---------------------------------------------------------------------------------------------
// KV pages: a free list on the host; the device page table is patched with small copies.
// Both models index positions the same way, so one page table serves both caches.
// ---------------------------------------------------------------------------------------------
int ensure_pages(stairs_ctx* ctx, int slot, int n_tokens) {
  const int pt = ctx->cfg.kv_page_tokens;
  const int need = (n_tokens + pt - 1) / pt;
  auto& pg = ctx->pages[slot];
  if ((int)pg.size() >= need) return STAIRS_OK;
  if (need > ctx->lay.max_pages) return fail(ctx, STAIRS_ENOSPC, "request %d would exceed max_seq_len", slot);
  const int first_new = (int)pg.size();
  if ((int)ctx->free_pages.size() < need - first_new)
    return fail(ctx, STAIRS_ENOSPC, "KV page pool exhausted (%d pages)", ctx->lay.n_pages);
  while ((int)pg.size() < need) { pg.push_back(ctx->free_pages.back()); ctx->free_pages.pop_back(); }
  int* dst = reinterpret_cast<int*>(ctx->ws + ctx->lay.page_table) + (size_t)slot * ctx->lay.max_pages + first_new;
  CK(cudaMemcpyAsync(dst, pg.data() + first_new, (size_t)(need - first_new) * 4, cudaMemcpyHostToDevice, ctx->stream));
  return STAIRS_OK;
}

void release_pages(stairs_ctx* ctx, int slot) {
  for (int p : ctx->pages[slot]) ctx->free_pages.push_back(p);
  ctx->pages[slot].clear();
  ctx->active[slot] = 0;
  ctx->n_seq_ub[slot] = 0;
}

// ---------------------------------------------------------------------------------------------
// Tensor-core GEMM plumbing: tensor maps and job set-up.
// ---------------------------------------------------------------------------------------------
// 2-D map of a row-major bf16 matrix [rows, K]; box = 64 k-elements x box_rows rows, 128-byte swizzle.
bool encode_map(stairs_ctx* ctx, CUtensorMap* out, const void* ptr, long long rows, long long K, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {(cuuint32_t)tc::BK, (cuuint32_t)box_rows};
  cuuint32_t es[2] = {1, 1};
  CUresult r = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// 3-D view of the same matrix for the persistent kernel: [K / 64][rows][64], box = 64 k-elements x
// box_rows rows x kps k-blocks, 128-byte swizzle: one copy brings kps consecutive K-major slabs.
bool encode_map3(stairs_ctx* ctx, CUtensorMap* out, const void* ptr, long long rows, long long K, int box_rows, int kps) {
  cuuint64_t dims[3] = {(cuuint64_t)tc::BK, (cuuint64_t)rows, (cuuint64_t)(K / tc::BK)};
  cuuint64_t strides[2] = {(cuuint64_t)K * 2, (cuuint64_t)tc::BK * 2};
  cuuint32_t box[3] = {(cuuint32_t)tc::BK, (cuuint32_t)box_rows, (cuuint32_t)kps};
  cuuint32_t es[3] = {1, 1, 1};
  CUresult r = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// One layer's K or V pool [pool rows, Hkv * hd] fp16: box = 64 columns (one 128-byte swizzle row) x
// box_rows rows (a page, or 64 rows of a larger page).
bool encode_kv_map(stairs_ctx* ctx, CUtensorMap* out, const void* ptr, long long pool_rows, int nkv, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)nkv, (cuuint64_t)pool_rows};
  cuuint64_t strides[1] = {(cuuint64_t)nkv * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  cuuint32_t es[2] = {1, 1};
  CUresult r = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

int build_weight_maps(stairs_ctx* ctx, DevModel& M) {
  const stairs_model& m = M.m;
  const int nq = m.n_heads * m.head_dim, nkv = m.n_kv_heads * m.head_dim;
  M.maps.resize(m.n_layers);
  bool ok = true;
  for (int l = 0; l < m.n_layers && ok; ++l) {
    const stairs_layer_w& w = M.layers[l];
    LayerMaps& t = M.maps[l];
    ok = ok && encode_map(ctx, &t.wq, w.wq, nq, m.d_model, tc::BM);
    ok = ok && encode_map(ctx, &t.wk, w.wk, nkv, m.d_model, tc::BM);
    ok = ok && encode_map(ctx, &t.wv, w.wv, nkv, m.d_model, tc::BM);
    ok = ok && encode_map(ctx, &t.wo, w.wo, m.d_model, nq, tc::BM);
    if (m.act == 1) {
      ok = ok && encode_map(ctx, &t.w1, w.w_gate_or_fc1, m.d_ff, m.d_model, 64);
      ok = ok && encode_map(ctx, &t.w3, w.w_up, m.d_ff, m.d_model, 64);
    } else {
      ok = ok && encode_map(ctx, &t.w1, w.w_gate_or_fc1, m.d_ff, m.d_model, tc::BM);
    }
    ok = ok && encode_map(ctx, &t.w2, w.w_down_or_fc2, m.d_model, m.d_ff, tc::BM);
  }
  ok = ok && encode_map(ctx, &M.head_map, M.w.lm_head, m.vocab, m.d_model, tc::BM);
  if (!ok) return fail(ctx, STAIRS_ECUDA, "cuTensorMapEncodeTiled failed for a weight matrix");
  return STAIRS_OK;
}

struct TcArgs {
  const CUtensorMap* w[3] = {nullptr, nullptr, nullptr};
  int rows[3] = {0, 0, 0};   // output features of each source
  int n_src = 1;
  bool dual = false;         // w[0] = gate, w[1] = up; rows[0] = d_ff
  const void* x = nullptr;   // activations [*, K] bf16
  int K = 0, T = 0;
  int epi = tc::TC_STORE_F32;
  float* out_f32 = nullptr; int ldo = 0;
  bf16* out_act = nullptr;
  unsigned long long* keys = nullptr;
};

int launch_gemm_tc(stairs_ctx* ctx, const TcArgs& a) {
  tc::GemmJob job;
  memset(&job, 0, sizeof job);
  const Layout& L = ctx->lay;
  job.t_tiles = (a.T + 255) / 256;
  job.t_box = ((a.T + job.t_tiles - 1) / job.t_tiles + 15) / 16 * 16;
  job.kblocks = (a.K + tc::BK - 1) / tc::BK;
  job.dual = a.dual ? 1 : 0;
  job.n_src = a.n_src;
  int col = 0, tiles = 0;
  if (a.dual) {
    job.w_map[0] = *a.w[0]; job.w_map[1] = *a.w[1]; job.w_map[2] = *a.w[0];
    job.N = a.rows[0];
    tiles = (a.rows[0] + 63) / 64;
    job.src_tiles[0] = tiles;
  } else {
    for (int s = 0; s < 3; ++s) {
      job.w_map[s] = *a.w[s < a.n_src ? s : 0];
      if (s < a.n_src) {
        job.src_tiles[s] = (a.rows[s] + tc::BM - 1) / tc::BM;
        job.src_col[s] = col;
        col += a.rows[s];
        tiles += job.src_tiles[s];
      }
    }
    job.N = col;
  }
  job.n_tiles = tiles;
  job.T = a.T;
  if (job.t_box > L.t_box_max || (long long)tiles * job.t_tiles > TC_COUNTERS)
    return fail(ctx, STAIRS_EUNSUPPORTED, "GEMM shape outside the tensor-core path's scratch");
  auto key = std::make_tuple(a.x, a.K, job.t_box);
  auto it = ctx->act_maps.find(key);
  if (it == ctx->act_maps.end()) {
    CUtensorMap mp;
    if (!encode_map(ctx, &mp, a.x, L.max_rows, a.K, job.t_box))
      return fail(ctx, STAIRS_ECUDA, "cuTensorMapEncodeTiled failed for an activation buffer");
    it = ctx->act_maps.emplace(key, mp).first;
  }
  job.x_map = it->second;
  job.stages = tc::pick_stages(job.t_box);
  job.epi = a.epi;
  job.out_f32 = a.out_f32; job.ldo = a.ldo; job.out_act = a.out_act; job.keys = a.keys;
  job.partial = reinterpret_cast<float*>(ctx->ws + L.gemm_partial);
  job.counters = reinterpret_cast<int*>(ctx->ws + L.gemm_counters);
  job.status = ctx->status_dev;
  job.wait_limit = ctx->wait_limit;
  const long long total = (long long)tiles * job.t_tiles * job.kblocks;
  const int grid = (int)std::min<long long>(std::min(ctx->sm_count, TC_GRID_MAX), total);
  tc::k_gemm_tc<<<grid, tc::THREADS, tc::smem_bytes(job.t_box, job.stages), ctx->stream>>>(job);
  return STAIRS_OK;
}

// ---------------------------------------------------------------------------------------------
// Persistent forward kernel: per (model, row box) program and launch.
// ---------------------------------------------------------------------------------------------
// u[n] = sum_k W[n,k] * g[k],  c[n] = sum_k W[n,k] * b[k]   (one warp per row, fp32)
__global__ void k_ln_aux(const bf16* __restrict__ W, const float* __restrict__ g, const float* __restrict__ b,
                         float* __restrict__ u, float* __restrict__ c, int N, int K) {
  const int n = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (n >= N) return;
  float su = 0.f, sc = 0.f;
  for (int k = lane; k < K; k += 32) {
    const float w = __bfloat162float(W[(size_t)n * K + k]);
    su = fmaf(w, g[k], su);
    sc = fmaf(w, b[k], sc);
  }
  su = warp_sum(su); sc = warp_sum(sc);
  if (lane == 0) { u[n] = su; c[n] = sc; }
}

// out[(128 t + j), :] = gate[64 t + j, :] and out[(128 t + 64 + j), :] = up[64 t + j, :] for j < 64
// (rows past d_ff are zero): every 128-row tile of `out` holds 64 gate rows and the matching 64 up
// rows, which is the shape the SwiGLU epilogue of the persistent kernel works on.
__global__ void k_pack_gate_up(const bf16* __restrict__ gate, const bf16* __restrict__ up, bf16* __restrict__ out, int F, int d) {
  const int row = blockIdx.x;                      // row of `out`
  const int t = row >> 7, j = row & 127;
  const int src_row = t * 64 + (j & 63);
  const bf16* src = (j < 64 ? gate : up) + (size_t)src_row * d;
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  for (int i = threadIdx.x; i < d / 8; i += blockDim.x)
    reinterpret_cast<uint4*>(out + (size_t)row * d)[i] = src_row < F ? reinterpret_cast<const uint4*>(src)[i] : zero;
}

// One-time per model: rotary frequency table, the interleaved gate/up matrices of SwiGLU models
// and, for LayerNorm models, the u/c vectors.
int setup_mk_model(stairs_ctx* ctx, DevModel& M, size_t rope_off, size_t aux_off, size_t w13_off, const DevModel* other) {
  const stairs_model& m = M.m;
  if (m.act == 1) {
    M.w13 = reinterpret_cast<bf16*>(ctx->ws + w13_off);
    const int rows = (m.d_ff + 63) / 64 * 128;
    M.w13_layer = (size_t)rows * m.d_model;
    M.w13_ptr.assign(m.n_layers, nullptr);
    for (int l = 0; l < m.n_layers; ++l) {
      // an early-exit assistant whose layer is one of the other model's layers shares its packed copy
      const bf16* shared = nullptr;
      if (other && other->w13)
        for (int j = 0; j < other->m.n_layers && !shared; ++j)
          if (other->layers[j].w_gate_or_fc1 == M.layers[l].w_gate_or_fc1 && other->layers[j].w_up == M.layers[l].w_up &&
              other->m.d_ff == m.d_ff)
            shared = other->w13_ptr[j];
      if (shared) { M.w13_ptr[l] = shared; continue; }
      bf16* dst = M.w13 + (size_t)l * M.w13_layer;
      k_pack_gate_up<<<rows, 128, 0, ctx->stream>>>((const bf16*)M.layers[l].w_gate_or_fc1, (const bf16*)M.layers[l].w_up, dst, m.d_ff, m.d_model);
      M.w13_ptr[l] = dst;
    }
    CK(cudaGetLastError());
  }
  M.rope_inv = reinterpret_cast<float*>(ctx->ws + rope_off);
  std::vector<float> inv(std::max(m.head_dim / 2, 1));
  for (int i = 0; i < m.head_dim / 2; ++i)
    inv[i] = (float)exp2(-(double)(2 * i) / (double)m.head_dim * log2((double)m.rope_theta));
  CK(cudaMemcpyAsync(M.rope_inv, inv.data(), (size_t)(m.head_dim / 2) * 4, cudaMemcpyHostToDevice, ctx->stream));
  CK(cudaStreamSynchronize(ctx->stream));
  if (m.norm != 0) return STAIRS_OK;
  M.ln_aux = reinterpret_cast<float*>(ctx->ws + aux_off);
  const int d = m.d_model, nq = m.n_heads * m.head_dim, nkv = m.n_kv_heads * m.head_dim, nqkv = nq + 2 * nkv, F = m.d_ff;
  const size_t f_aux = (size_t)F * (m.act == 1 ? 2 : 1);
  const size_t aux_layer = ((size_t)nqkv + f_aux) * 2;
  auto run = [&](const void* W, const void* g, const void* b, float* u, float* c, int N) {
    k_ln_aux<<<(N + 7) / 8, 256, 0, ctx->stream>>>((const bf16*)W, (const float*)g, (const float*)b, u, c, N, d);
  };
  for (int l = 0; l < m.n_layers; ++l) {
    const stairs_layer_w& w = M.layers[l];
    float* b2 = M.ln_aux + (size_t)l * aux_layer;
    float* qu = b2; float* qc = b2 + nqkv; float* fu = b2 + 2 * (size_t)nqkv; float* fc = fu + f_aux;
    run(w.wq, w.norm1_w, w.norm1_b, qu, qc, nq);
    run(w.wk, w.norm1_w, w.norm1_b, qu + nq, qc + nq, nkv);
    run(w.wv, w.norm1_w, w.norm1_b, qu + nq + nkv, qc + nq + nkv, nkv);
    run(w.w_gate_or_fc1, w.norm2_w, w.norm2_b, fu, fc, F);
    if (m.act == 1) run(w.w_up, w.norm2_w, w.norm2_b, fu + F, fc + F, F);
  }
  float* hu = M.ln_aux + (size_t)m.n_layers * aux_layer;
  run(M.w.lm_head, M.w.final_norm_w, M.w.final_norm_b, hu, hu + m.vocab, m.vocab);
  CK(cudaGetLastError());
  CK(cudaStreamSynchronize(ctx->stream));
  return STAIRS_OK;
}

// Shared-memory plan of the persistent kernel for one (model, row box): pipeline depth of the GEMM
// ring against the K/V chunk buffers of the attention phases.
struct MkPlan { int kps, stages, att_dbl, att_tma, att_nbuf, att_tc, att_qblk, att_q_rows; };

// q_rows_call: query rows (rows x grouped heads of the largest request, at most 128) of this call; 0 = the
// largest a call of this row box can have (the stage depth kps, which the programs' tensor maps carry,
// is decided for that case, so that it is the same for every call of the row box)
MkPlan mk_plan(const stairs_ctx* ctx, const stairs_model& m, int t_box, int q_rows_call = 0, int tc_call = -1) {
  MkPlan pl{};
  const int hd = m.head_dim;
  const int gq = m.n_heads / m.n_kv_heads;
  auto round8 = [](int v) { return (v + 7) / 8 * 8; };
  const int q_rows_max = std::min(mk::ATT_QBLK_TC, round8(t_box * gq));
  // copy path: two K/V chunk buffers where they are cheap (small heads) or needed (contexts so long
  // that a unit walks several chunks)
  pl.att_dbl = (hd <= 64 || (long long)ctx->cfg.max_seq_len * m.n_kv_heads / mk::ATT_CHUNK > 2ll * ctx->sm_count) ? 1 : 0;
  pl.att_tma = (ctx->att_tma_off == 0 && (hd == 64 || hd == 128)) ? 1 : 0;
  // tcgen05 attention: possible where the bulk-copy path is; used by the calls it pays for (tc_call, see
  // launch_forward_mk); tc_call < 0 plans for the mode that needs more shared memory
  const bool tc_possible = pl.att_tma && ctx->att_tc_off == 0;
  pl.att_tc = (tc_possible && tc_call != 0) ? 1 : 0;
  pl.att_qblk = pl.att_tc ? mk::ATT_QBLK_TC : mk::ATT_QBLK;
  pl.att_q_rows = pl.att_tc ? (q_rows_call > 0 ? std::min(q_rows_max, round8(q_rows_call)) : q_rows_max) : 0;
  // K/V chunk buffers wanted (bulk-copy paths): as many whole chunks as one SM's share of a layer's K/V
  // holds, at most four; the tcgen05 path wants two at least, so that a chunk loads while the previous
  // one is multiplied.  Measured: the GEMM ring matters more than chunk buffers, so a buffer beyond
  // the minimum is only added while the ring keeps three two-k-block stages (or four single ones).
  int want = 0, least = 0;
  if (pl.att_tma) {
    const long long kv_per_cta = (long long)ctx->cfg.max_requests * ctx->cfg.max_seq_len * m.n_kv_heads * hd * 4 / std::max(ctx->sm_count, 1);
    const long long chunk = (long long)mk::AttnSmem::kv_buf_bytes(hd);
    least = pl.att_tc ? 2 : 1;
    want = (int)std::min<long long>(mk::MAX_KV_BUF, std::max<long long>(least, kv_per_cta / chunk));
    if (ctx->att_nbuf_force > 0) want = least = std::min(ctx->att_nbuf_force, (int)mk::MAX_KV_BUF);
  }
  auto stages_for = [&](int kps, int nbuf) { return mk::pick_stages(t_box, hd, pl.att_dbl, kps, pl.att_tma, nbuf, pl.att_q_rows); };
  pl.kps = (ctx->kps_force > 0) ? ctx->kps_force : (stages_for(2, least) >= 3 ? 2 : 1);
  if (stages_for(pl.kps, least) < 2) pl.kps = 1;
  pl.att_nbuf = least;
  // (the tcgen05 path is used where attention dominates the call: there a third buffer is worth a fourth stage)
  while (pl.att_nbuf < want && stages_for(pl.kps, pl.att_nbuf + 1) >= ((pl.kps == 2 || (pl.att_tc && pl.att_nbuf < 3)) ? 3 : 4)) ++pl.att_nbuf;
  pl.stages = stages_for(pl.kps, pl.att_nbuf);
  return pl;
}


int build_program(stairs_ctx* ctx, DevModel& M, int t_box, int kps) {
  const stairs_model& m = M.m;
  const Layout& L = ctx->lay;
  const int slot = (t_box / 16 - 1) * 2 + (kps - 1);
  const int d = m.d_model, nq = m.n_heads * m.head_dim, nkv = m.n_kv_heads * m.head_dim, nqkv = nq + 2 * nkv, F = m.d_ff;
  char* ws = ctx->ws;
  std::vector<CUtensorMap> maps((size_t)9 * m.n_layers + 4);
  bool ok = true;
  for (int l = 0; l < m.n_layers && ok; ++l) {
    const stairs_layer_w& w = M.layers[l];
    CUtensorMap* b = &maps[(size_t)7 * l];
    ok = ok && encode_map3(ctx, &b[0], w.wq, nq, d, tc::BM, kps) && encode_map3(ctx, &b[1], w.wk, nkv, d, tc::BM, kps) &&
         encode_map3(ctx, &b[2], w.wv, nkv, d, tc::BM, kps) && encode_map3(ctx, &b[3], w.wo, d, nq, tc::BM, kps);
    if (m.act == 1) ok = ok && encode_map3(ctx, &b[4], M.w13_ptr[l], (F + 63) / 64 * 128, d, tc::BM, kps);
    else ok = ok && encode_map3(ctx, &b[4], w.w_gate_or_fc1, F, d, tc::BM, kps);
    b[5] = b[4];
    ok = ok && encode_map3(ctx, &b[6], w.w_down_or_fc2, d, F, tc::BM, kps);
  }
  const int i_head = 7 * m.n_layers, i_h = i_head + 1, i_o = i_head + 2, i_ff = i_head + 3;
  ok = ok && encode_map3(ctx, &maps[i_head], M.w.lm_head, m.vocab, d, tc::BM, kps);
  // activation operands: the lo parts' rows follow the hi parts' t_box rows, so one box of
  // 2 * t_box rows brings both
  ok = ok && encode_map3(ctx, &maps[i_h], ws + L.h, 2 * L.max_rows, d, 2 * t_box, kps) &&
       encode_map3(ctx, &maps[i_o], ws + L.o, 2 * L.max_rows, nq, 2 * t_box, kps) &&
       encode_map3(ctx, &maps[i_ff], ws + L.ff, 2 * L.max_rows, F, 2 * t_box, kps);
  // K/V pools of every layer, for the attention phases' bulk copies
  const int i_kv = i_head + 4;
  const int kv_box_rows = std::min(ctx->cfg.kv_page_tokens, mk::ATT_CHUNK);
  const long long pool_rows = (long long)L.n_pages * ctx->cfg.kv_page_tokens;
  if (m.head_dim % 64 == 0)
    for (int l = 0; l < m.n_layers && ok; ++l)
      ok = ok && encode_kv_map(ctx, &maps[i_kv + 2 * l], M.kpool + (size_t)l * M.kv_layer_bytes, pool_rows, nkv, kv_box_rows) &&
           encode_kv_map(ctx, &maps[i_kv + 2 * l + 1], M.vpool + (size_t)l * M.kv_layer_bytes, pool_rows, nkv, kv_box_rows);
  if (!ok) return fail(ctx, STAIRS_ECUDA, "cuTensorMapEncodeTiled failed for a weight matrix, an activation buffer or a K/V pool");
  std::vector<mk::Phase> ph;
  auto gemm = [&](int layer, int w0, int w1, int w2, int n_src, const int* rows, bool dual, int xmap, int K, int epi, void* out, int ldo) -> mk::Phase& {
    mk::Phase p;
    memset(&p, 0, sizeof p);
    p.kind = mk::PH_GEMM; p.layer = layer;
    p.w_map[0] = w0; p.w_map[1] = w1; p.w_map[2] = w2; p.x_map = xmap;
    p.n_src = n_src; p.dual = dual ? 1 : 0;
    p.kblocks = ((K + tc::BK - 1) / tc::BK + kps - 1) / kps;   // pipeline stages (groups of kps k-blocks) per tile
    p.upt = ((K + tc::BK - 1) / tc::BK + mk::RANGE_UNIT_KB - 1) / mk::RANGE_UNIT_KB;
    int col = 0, tiles = 0;
    if (dual) { p.N = rows[0]; tiles = (rows[0] + 63) / 64; p.src_tiles[0] = tiles; }
    else {
      for (int s2 = 0; s2 < n_src; ++s2) {
        p.src_tiles[s2] = (rows[s2] + tc::BM - 1) / tc::BM; p.src_col[s2] = col; col += rows[s2]; tiles += p.src_tiles[s2];
      }
      p.N = col;
    }
    p.n_tiles = tiles; p.epi = epi; p.out = out; p.ldo = ldo;
    {
      // How many CTAs to cut this GEMM over: more CTAs stream faster, but every tile is then
      // finished from more partial tiles, which the finisher reads four at a time.  Model:
      // stream time at ~44 GB/s per SM plus ~1.6 us per batch of four partials.
      const int grid = std::min(ctx->sm_count, TC_GRID_MAX);
      const double bytes = (double)tiles * ((K + tc::BK - 1) / tc::BK) * tc::A_STAGE_BYTES;   // (must not depend on the row box: see RANGE_UNIT_KB)
      double best = 1e30; int best_ge = grid;
      for (int s2 = 1; s2 <= 64; s2 *= 2) {
        const int ge = std::min(grid, tiles * s2);
        const double seg = (double)ge / tiles + (ge % tiles ? 1.0 : 0.0);
        const double t_us = bytes / (ge * 44.0e3) + (seg > 1.0 ? std::ceil(seg / 4.0) * 1.6 + 2.0 : 0.0);
        if (t_us < best - 1e-9) { best = t_us; best_ge = ge; }
        if (ge == grid) break;
      }
      p.ge_max = best_ge;
    }
    ph.push_back(p);
    return ph.back();
  };
  auto simple = [&](int kind, int layer, const void* g, void* kc, void* vc) {
    mk::Phase p;
    memset(&p, 0, sizeof p);
    p.kind = kind; p.layer = layer; p.g = (const float*)g; p.kc = kc; p.vc = vc;
    ph.push_back(p);
  };
  // LayerNorm auxiliary vectors, laid out per layer as [qkv u | qkv c | mlp u | mlp c], then [head u | head c]
  const bool ln = m.norm == 0;
  const size_t f_aux = (size_t)F * (m.act == 1 ? 2 : 1);
  const size_t aux_layer = ((size_t)nqkv + f_aux) * 2;
  auto aux_ptr = [&](int l, int which) -> const float* {   // which: 0 qkv u, 1 qkv c, 2 mlp u, 3 mlp c
    if (!ln) return nullptr;
    const float* b2 = M.ln_aux + (size_t)l * aux_layer;
    if (which == 0) return b2;
    if (which == 1) return b2 + nqkv;
    if (which == 2) return b2 + 2 * (size_t)nqkv;
    return b2 + 2 * (size_t)nqkv + f_aux;
  };
  simple(mk::PH_EMBED, 0, M.layers[0].norm1_w, nullptr, nullptr);
  for (int l = 0; l < m.n_layers; ++l) {
    const stairs_layer_w& w = M.layers[l];
    const int b = 7 * l;
    const int r3[3] = {nq, nkv, nkv};
    const bool in_epilogue = m.pos == 0 || m.head_dim == 64 || m.head_dim == 128;
    {
      mk::Phase& p = gemm(l, b + 0, b + 1, b + 2, 3, r3, false, i_h, d, tc::TC_STORE_F32, ws + L.qkv, nqkv);
      p.norm_in = 1; p.u = aux_ptr(l, 0); p.c = aux_ptr(l, 1);
      // q to the query buffer, k and v (fp16) to this layer's cache rows: in the epilogue where a
      // rotation pair sits in one thread (head size 64 or 128, or no rotation), else in a phase of its own
      p.qkv_prep = in_epilogue ? 1 : 0;
      p.kc = M.kpool + (size_t)l * M.kv_layer_bytes; p.vc = M.vpool + (size_t)l * M.kv_layer_bytes;
    }
    if (!in_epilogue) simple(mk::PH_PREP, l, nullptr, M.kpool + (size_t)l * M.kv_layer_bytes, M.vpool + (size_t)l * M.kv_layer_bytes);
    simple(mk::PH_ATTN, l, nullptr, M.kpool + (size_t)l * M.kv_layer_bytes, M.vpool + (size_t)l * M.kv_layer_bytes);
    ph.back().w_map[0] = i_kv + 2 * l; ph.back().w_map[1] = i_kv + 2 * l + 1;   // the layer's K and V pool maps
    const int rd[1] = {d};
    {
      mk::Phase& p = gemm(l, b + 3, b + 3, b + 3, 1, rd, false, i_o, nq, tc::TC_ADD_F32, ws + L.x, d);
      p.next_g = (const float*)w.norm2_w;
    }
    const int rf[1] = {F};
    {
      mk::Phase& p = (m.act == 1) ? gemm(l, b + 4, b + 4, b + 4, 1, rf, true, i_h, d, tc::TC_SWIGLU, ws + L.ff, F)
                                  : gemm(l, b + 4, b + 4, b + 4, 1, rf, false, i_h, d, tc::TC_GELU, ws + L.ff, F);
      p.norm_in = 1; p.u = aux_ptr(l, 2); p.c = aux_ptr(l, 3);
    }
    {
      mk::Phase& p = gemm(l, b + 6, b + 6, b + 6, 1, rd, false, i_ff, F, tc::TC_ADD_F32, ws + L.x, d);
      p.next_g = (const float*)(l + 1 < m.n_layers ? M.layers[l + 1].norm1_w : M.w.final_norm_w);
    }
  }
  {
    const int rv[1] = {m.vocab};
    mk::Phase& p = gemm(-1, i_head, i_head, i_head, 1, rv, false, i_h, d, tc::TC_LMHEAD, nullptr, m.vocab);
    p.norm_in = 1;
    if (ln) { p.u = M.ln_aux + (size_t)m.n_layers * aux_layer; p.c = p.u + m.vocab; }
  }
  simple(mk::PH_ACCEPT, -1, nullptr, nullptr, nullptr);
  for (const mk::Phase& p : ph)
    if (p.kind == mk::PH_GEMM && (p.n_tiles > TC_COUNTERS || (long long)p.n_tiles * p.kblocks * TC_GRID_MAX >= (1ll << 32)))
      return fail(ctx, STAIRS_EUNSUPPORTED, "too many tiles for the split bookkeeping");
  M.n_phases = (int)ph.size();
  char* base = M.prog_base + (size_t)slot * M.prog_slot_bytes;
  if (ph.size() * sizeof(mk::Phase) > M.prog_maps_off || M.prog_maps_off + maps.size() * sizeof(CUtensorMap) > M.prog_slot_bytes)
    return fail(ctx, STAIRS_ENOSPC, "program area too small");
  CK(cudaMemcpyAsync(base, ph.data(), ph.size() * sizeof(mk::Phase), cudaMemcpyHostToDevice, ctx->stream));
  CK(cudaMemcpyAsync(base + M.prog_maps_off, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, ctx->stream));
  CK(cudaStreamSynchronize(ctx->stream));   // the host vectors go away
  M.prog_built[slot] = true;
  return STAIRS_OK;
}

struct MkCall {
  int mode = mk::CALL_VALIDATE, n_req = 0, slot = 0, draft_step = 0;
  const int* draft = nullptr;
  int* target_tokens = nullptr; int* accept_len = nullptr; int commit = 0; int* draft_out = nullptr;
  float* logits = nullptr;
  bool skip_head = false;   // prefill: stop after the last layer (no LM head, no accept)
  const int* req_host = nullptr; // validate: slot, draft length and first row per request (travel as kernel parameters)
  const int* k_host = nullptr;
  const int* off_host = nullptr;
};

bool mk_eligible(const stairs_ctx* ctx, const DevModel& M, int T) {
  // (the epilogue's vector stores want every GEMM width but the vocabulary to be a multiple of 4)
  return ctx->use_mk && M.m.n_layers >= 1 && T >= 1 && T <= MK_MAX_ROWS && M.m.head_dim % 16 == 0 && M.m.head_dim <= 128 &&
         M.m.d_model % 64 == 0 && M.m.d_ff % 64 == 0 && (M.m.n_heads * M.m.head_dim) % 64 == 0 && M.m.d_model <= 8192;
}

int launch_forward_mk(stairs_ctx* ctx, DevModel& M, int T, int logit_first_row, int n_logit_rows, const MkCall& c) {
  const stairs_model& m = M.m;
  const Layout& L = ctx->lay;
  char* ws = ctx->ws;
  const int t_box = (T + 15) / 16 * 16;
  int q_rows_call = 0, tc_call = 0;
  long long units_avail = 0;
  {
    // attention scratch: refuse a call whose units might not fit rather than compute part of it
    const int hkv = m.n_kv_heads, gq = m.n_heads / m.n_kv_heads;
    long long need = 0;
    // The tcgen05 attention path pays where a unit walks many chunks (long contexts) or a request has
    // many query rows (prefill passes: 128 queries share a chunk instead of 48); short units are
    // quicker on the register path, whose per-unit set-up is smaller.
    int r_max0 = 0; long long len_max = 0;
    if (c.mode == mk::CALL_VALIDATE) for (int i = 0; i < c.n_req; ++i) { r_max0 = std::max(r_max0, c.k_host[i] + 1); len_max = std::max<long long>(len_max, ctx->n_seq_ub[c.req_host[i]]); }
    else { r_max0 = T; len_max = c.mode == mk::CALL_PREFILL ? c.draft_step + T : ctx->n_seq_ub[c.slot]; }
    const long long chunks_per_unit = (len_max / mk::ATT_CHUNK + 1) * hkv / std::max(ctx->sm_count, 1);
    // (with many query rows its tiles take shared memory from the GEMM ring: only past a few thousand positions)
    tc_call = (ctx->att_tc_force > 0 || chunks_per_unit >= 6 || (r_max0 * gq >= 96 && len_max >= 4096)) ? 1 : 0;
    const MkPlan pl0 = mk_plan(ctx, m, t_box, 0, tc_call);
    int r_max = 0;
    if (c.mode == mk::CALL_VALIDATE) for (int i = 0; i < c.n_req; ++i) { need += attn_unit_bound(hkv, gq, c.k_host[i] + 1, pl0.att_qblk); r_max = std::max(r_max, c.k_host[i] + 1); }
    else { need = attn_unit_bound(hkv, gq, T, pl0.att_qblk); r_max = T; }
    q_rows_call = std::min(r_max * gq, (int)mk::ATT_QBLK_TC);
    units_avail = (long long)(L.attn_part_bytes / ((size_t)pl0.att_qblk * (m.head_dim + 4) * 4));
    if (need > units_avail)
      return fail(ctx, STAIRS_ENOSPC, "attention scratch holds %lld units, this call may need %lld", units_avail, need);
  }
  const MkPlan pl = mk_plan(ctx, m, t_box, q_rows_call, tc_call);
  const int slot = (t_box / 16 - 1) * 2 + (pl.kps - 1);
  if (!M.prog_built[slot]) {
    int rc = build_program(ctx, M, t_box, pl.kps);
    if (rc) return rc;
  }
  mk::Params P;
  memset(&P, 0, sizeof P);
  char* base = M.prog_base + (size_t)slot * M.prog_slot_bytes;
  const int n_run = c.skip_head ? M.n_phases - 2 : M.n_phases;
  P.phases = reinterpret_cast<const mk::Phase*>(base); P.n_phases = n_run;
  P.maps = reinterpret_cast<const CUtensorMap*>(base + M.prog_maps_off);
  P.T = T; P.t_box = t_box;
  P.att_dbl = pl.att_dbl; P.att_tma = pl.att_tma; P.att_nbuf = pl.att_nbuf;
  P.att_tc = pl.att_tc; P.att_qblk = pl.att_qblk; P.att_q_rows = pl.att_q_rows;
  P.kv_box_rows = std::min(ctx->cfg.kv_page_tokens, mk::ATT_CHUNK);
  P.kps = pl.kps;
  P.stages = pl.stages;
  P.logit_first_row = logit_first_row; P.n_logit_rows = n_logit_rows;
  P.d = m.d_model; P.Hq = m.n_heads; P.Hkv = m.n_kv_heads; P.hd = m.head_dim; P.F = m.d_ff; P.vocab = m.vocab;
  P.norm_kind = m.norm; P.rope = m.pos; P.rope_theta = m.rope_theta; P.eps = m.norm_eps;
  P.tok_emb = (const bf16*)M.w.tok_emb; P.pos_emb = (const bf16*)M.w.pos_emb;
  P.mode = c.mode; P.n_req = c.n_req; P.slot = c.slot; P.draft_step = c.draft_step;
  P.draft_first_rows = ctx->draft_shares_kv ? 1 : 2;
  if (c.mode == mk::CALL_VALIDATE)
    for (int i = 0; i < c.n_req; ++i) { P.val_req[i] = c.req_host[i]; P.val_k[i] = c.k_host[i]; P.val_off[i] = c.off_host[i]; }
  P.draft = c.draft; P.k_max = ctx->cfg.k_max;
  P.seq = reinterpret_cast<int*>(ws + L.seq); P.n_seq = reinterpret_cast<int*>(ws + L.n_seq); P.max_seq_len = ctx->cfg.max_seq_len;
  P.tok = reinterpret_cast<int*>(ws + L.tok); P.pos = reinterpret_cast<int*>(ws + L.pos); P.req = reinterpret_cast<int*>(ws + L.req);
  P.page_table = reinterpret_cast<int*>(ws + L.page_table); P.page_tokens = ctx->cfg.kv_page_tokens; P.max_pages = L.max_pages;
  P.x = reinterpret_cast<float*>(ws + L.x); P.h = reinterpret_cast<bf16*>(ws + L.h); P.qkv = reinterpret_cast<float*>(ws + L.qkv);
  P.q16 = reinterpret_cast<__half*>(ws + L.q);
  P.o = reinterpret_cast<bf16*>(ws + L.o); P.ff = reinterpret_cast<bf16*>(ws + L.ff);
  P.lo_row = t_box;   // lo parts directly after the hi parts of this launch's row box
  P.keys = reinterpret_cast<unsigned long long*>(ws + L.keys); P.n_keys = L.max_rows;
  P.logits = c.logits;
  P.target_tokens = c.target_tokens; P.accept_len = c.accept_len; P.commit = c.commit; P.draft_out = c.draft_out;
  P.partial = reinterpret_cast<float*>(ws + L.mk_partial); P.counters = reinterpret_cast<int*>(ws + L.gemm_counters);
  P.attn_part = reinterpret_cast<float*>(ws + L.attn_part); P.attn_part_units = (int)units_avail;
  P.attn_set_stride = L.attn_part_bytes / 4;
  P.stats = reinterpret_cast<float4*>(ws + L.mk_stats); P.stat_tiles = L.stat_tiles;
  P.rope_inv = M.rope_inv; P.rope_cs = M.rope_inv + m.head_dim / 2; P.rope_sn = P.rope_cs + 64 * (m.head_dim / 2);
  P.bar = reinterpret_cast<unsigned long long*>(ws + L.mk_bar); P.bar_base = ctx->bar_base;
  P.status = ctx->status_dev; P.wait_limit = ctx->wait_limit;
  P.trace = (ctx->profile && &M == &ctx->target) ? reinterpret_cast<unsigned long long*>(ws + L.mk_trace) : nullptr;
  const int grid = std::min(ctx->sm_count, TC_GRID_MAX);
  void* args[] = {&P};
  CK(cudaLaunchCooperativeKernel((const void*)mk::k_forward, dim3(grid), dim3(mk::MK_THREADS), args,
                                 mk::smem_bytes(t_box, P.stages, m.head_dim, P.att_dbl, P.kps, P.att_tma, P.att_nbuf, P.att_q_rows), ctx->stream));
  ctx->bar_base += (unsigned long long)n_run * grid;
  ctx->launches++;
  return STAIRS_OK;
}

// ---------------------------------------------------------------------------------------------
// One forward pass over T rows (tok/pos/req already built on the device).
// ---------------------------------------------------------------------------------------------
struct GemmTimer {
  stairs_ctx* c;
  bool on;
  explicit GemmTimer(stairs_ctx* ctx)
      : c(ctx), on(ctx->profile && ctx->in_validate && ctx->ev_used + 2 <= (int)ctx->ev.size()) {
    if (on) cudaEventRecord(c->ev[c->ev_used++], c->stream);
  }
  ~GemmTimer() { if (on) cudaEventRecord(c->ev[c->ev_used++], c->stream); }
};

template <typename WT>
int forward_rows(stairs_ctx* ctx, DevModel& M, int T, int logit_first_row, int n_logit_rows, float* logits_out) {
  const stairs_model& m = M.m;
  const Layout& L = ctx->lay;
  cudaStream_t st = ctx->stream;
  char* ws = ctx->ws;
  const int d = m.d_model, hq = m.n_heads, hkv = m.n_kv_heads, hd = m.head_dim, F = m.d_ff;
  const int nq = hq * hd, nkv = hkv * hd, nqkv = nq + 2 * nkv;
  const int* tok = reinterpret_cast<int*>(ws + L.tok);
  const int* pos = reinterpret_cast<int*>(ws + L.pos);
  const int* req = reinterpret_cast<int*>(ws + L.req);
  const int* page_table = reinterpret_cast<int*>(ws + L.page_table);
  float* x = reinterpret_cast<float*>(ws + L.x);
  WT* h = reinterpret_cast<WT*>(ws + L.h);
  float* qkv = reinterpret_cast<float*>(ws + L.qkv);
  WT* q = reinterpret_cast<WT*>(ws + L.q);
  WT* o = reinterpret_cast<WT*>(ws + L.o);
  WT* ff = reinterpret_cast<WT*>(ws + L.ff);
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(ws + L.keys);
  const int pt = ctx->cfg.kv_page_tokens;

  constexpr bool kBf16 = std::is_same<WT, bf16>::value;
  const bool use_tc = kBf16 && ctx->use_tc;
  int rc = STAIRS_OK;
  k_embed<WT><<<T, 256, 0, st>>>((const WT*)M.w.tok_emb, (const WT*)M.w.pos_emb, tok, pos, x, d);
  ctx->launches++;
  for (int l = 0; l < m.n_layers && !rc; ++l) {
    const stairs_layer_w& w = M.layers[l];
    typedef typename KvType<WT>::type KT;
    KT* kc = reinterpret_cast<KT*>(M.kpool + (size_t)l * M.kv_layer_bytes);
    KT* vc = reinterpret_cast<KT*>(M.vpool + (size_t)l * M.kv_layer_bytes);
    k_norm<WT><<<T, 256, 0, st>>>(x, (const float*)w.norm1_w, (const float*)w.norm1_b, h, d, m.norm, m.norm_eps);
    {
      GemmTimer tm(ctx);
      if (use_tc) {
        TcArgs a;
        a.w[0] = &M.maps[l].wq; a.w[1] = &M.maps[l].wk; a.w[2] = &M.maps[l].wv;
        a.rows[0] = nq; a.rows[1] = nkv; a.rows[2] = nkv; a.n_src = 3;
        a.x = h; a.K = d; a.T = T; a.epi = tc::TC_STORE_F32; a.out_f32 = qkv; a.ldo = nqkv;
        rc = launch_gemm_tc(ctx, a);
        ctx->launches += 1;
      } else {
        launch_gemm_rows<WT, false>(st, (const WT*)w.wq, nullptr, h, T, nq, d, EPI_STORE_F32, qkv, nullptr, nqkv);
        launch_gemm_rows<WT, false>(st, (const WT*)w.wk, nullptr, h, T, nkv, d, EPI_STORE_F32, qkv + nq, nullptr, nqkv);
        launch_gemm_rows<WT, false>(st, (const WT*)w.wv, nullptr, h, T, nkv, d, EPI_STORE_F32, qkv + nq + nkv, nullptr, nqkv);
        ctx->launches += 3;
      }
    }
    if (rc) break;
    k_rope_append<WT, KT><<<T, 256, 0, st>>>(qkv, pos, req, page_table, q, kc, vc, hq, hkv, hd, m.pos, m.rope_theta, pt, L.max_pages);
    k_attn_plain<WT, KT, 8><<<dim3(hq, T), 128, (size_t)5 * hd * sizeof(float), st>>>(
        q, kc, vc, page_table, req, pos, o, hq, hkv, hd, pt, L.max_pages, 1.0f / sqrtf((float)hd));
    {
      GemmTimer tm(ctx);
      if (use_tc) {
        TcArgs a;
        a.w[0] = &M.maps[l].wo; a.rows[0] = d; a.x = o; a.K = nq; a.T = T;
        a.epi = tc::TC_ADD_F32; a.out_f32 = x; a.ldo = d;
        rc = launch_gemm_tc(ctx, a);
      } else {
        launch_gemm_rows<WT, false>(st, (const WT*)w.wo, nullptr, o, T, d, nq, EPI_ADD_F32, x, nullptr, d);
      }
    }
    if (rc) break;
    k_norm<WT><<<T, 256, 0, st>>>(x, (const float*)w.norm2_w, (const float*)w.norm2_b, h, d, m.norm, m.norm_eps);
    {
      GemmTimer tm(ctx);
      if (use_tc) {
        TcArgs a;
        a.w[0] = &M.maps[l].w1; a.rows[0] = F; a.x = h; a.K = d; a.T = T;
        a.out_act = reinterpret_cast<bf16*>(ff); a.ldo = F;
        if (m.act == 1) { a.w[1] = &M.maps[l].w3; a.dual = true; a.epi = tc::TC_SWIGLU; }
        else a.epi = tc::TC_GELU;
        rc = launch_gemm_tc(ctx, a);
        if (!rc) {
          TcArgs b;
          b.w[0] = &M.maps[l].w2; b.rows[0] = d; b.x = ff; b.K = F; b.T = T;
          b.epi = tc::TC_ADD_F32; b.out_f32 = x; b.ldo = d;
          rc = launch_gemm_tc(ctx, b);
        }
      } else {
        if (m.act == 1)
          launch_gemm_rows<WT, true>(st, (const WT*)w.w_gate_or_fc1, (const WT*)w.w_up, h, T, F, d, EPI_SWIGLU, nullptr, ff, F);
        else
          launch_gemm_rows<WT, false>(st, (const WT*)w.w_gate_or_fc1, nullptr, h, T, F, d, EPI_GELU, nullptr, ff, F);
        launch_gemm_rows<WT, false>(st, (const WT*)w.w_down_or_fc2, nullptr, ff, T, d, F, EPI_ADD_F32, x, nullptr, d);
      }
    }
    ctx->launches += 7;
  }
  if (rc) return rc;
  if (n_logit_rows > 0) {
    k_norm<WT><<<n_logit_rows, 256, 0, st>>>(x + (size_t)logit_first_row * d, (const float*)M.w.final_norm_w,
                                             (const float*)M.w.final_norm_b, h, d, m.norm, m.norm_eps);
    ctx->launches += 1;
    if (use_tc) {
      // LM head with the vocabulary argmax fused into the epilogue; logits are stored only on request
      GemmTimer tm(ctx);
      TcArgs a;
      a.w[0] = &M.head_map; a.rows[0] = m.vocab; a.x = h; a.K = d; a.T = n_logit_rows;
      a.epi = tc::TC_LMHEAD; a.out_f32 = logits_out; a.ldo = m.vocab; a.keys = keys + logit_first_row;
      rc = launch_gemm_tc(ctx, a);
      ctx->launches += 1;
      if (rc) return rc;
    } else {
      float* lg = logits_out ? logits_out : reinterpret_cast<float*>(ws + L.logits);
      {
        GemmTimer tm(ctx);
        launch_gemm_rows<WT, false>(st, (const WT*)M.w.lm_head, nullptr, h, n_logit_rows, m.vocab, d, EPI_STORE_F32, lg, nullptr, m.vocab);
      }
      const int slices = std::max(1, std::min(64, m.vocab / 2048));
      k_argmax<<<dim3(slices, n_logit_rows), 256, 0, st>>>(lg, m.vocab, m.vocab, keys + logit_first_row);
      ctx->launches += 2;
    }
  }
  CK(cudaGetLastError());
  return STAIRS_OK;
}

int forward(stairs_ctx* ctx, DevModel& M, int T, int logit_first_row, int n_logit_rows, float* logits_out) {
  if (M.m.wdtype == 0) return forward_rows<float>(ctx, M, T, logit_first_row, n_logit_rows, logits_out);
  return forward_rows<bf16>(ctx, M, T, logit_first_row, n_logit_rows, logits_out);
}

RowParams base_rows(stairs_ctx* ctx) {
  RowParams p{};
  char* ws = ctx->ws;
  const Layout& L = ctx->lay;
  p.val_req = reinterpret_cast<int*>(ws + L.val_req);
  p.val_k = reinterpret_cast<int*>(ws + L.val_k);
  p.val_off = reinterpret_cast<int*>(ws + L.val_off);
  p.k_max = ctx->cfg.k_max;
  p.seq = reinterpret_cast<int*>(ws + L.seq);
  p.n_seq = reinterpret_cast<int*>(ws + L.n_seq);
  p.max_seq_len = ctx->cfg.max_seq_len;
  p.vocab = ctx->cfg.target.vocab;
  p.tok = reinterpret_cast<int*>(ws + L.tok);
  p.pos = reinterpret_cast<int*>(ws + L.pos);
  p.req = reinterpret_cast<int*>(ws + L.req);
  p.keys = reinterpret_cast<unsigned long long*>(ws + L.keys);
  p.n_keys = L.max_rows;
  return p;
}

int launch_rows(stairs_ctx* ctx, const RowParams& p, int threads_needed) {
  const int n = std::max(threads_needed, p.n_keys);
  k_rows<<<(n + 255) / 256, 256, 0, ctx->stream>>>(p);
  ctx->launches++;
  CK(cudaGetLastError());
  return STAIRS_OK;
}

int check_slot(stairs_ctx* ctx, int req, bool must_be_active) {
  if (!ctx) return STAIRS_EINVAL;
  if (req < 0 || req >= ctx->cfg.max_requests) return fail(ctx, STAIRS_EINVAL, "request slot %d out of range", req);
  if (must_be_active && !ctx->active[req]) return fail(ctx, STAIRS_ESTATE, "request %d has not been prefilled", req);
  return STAIRS_OK;
}

int prefill_model(stairs_ctx* ctx, DevModel& M, int slot, int n_ctx) {
  if (mk_eligible(ctx, M, MK_MAX_ROWS)) {
    // through the persistent kernel, 64 positions per pass: same arithmetic (hi+lo operands,
    // fp16 attention tiles) as the validation pass, so cached K/V are as accurate as new ones
    for (int c0 = 0; c0 < n_ctx; c0 += MK_MAX_ROWS) {
      MkCall c;
      c.mode = mk::CALL_PREFILL; c.slot = slot; c.draft_step = c0; c.skip_head = true;
      int rc = launch_forward_mk(ctx, M, std::min(MK_MAX_ROWS, n_ctx - c0), 0, 0, c);
      if (rc) return rc;
    }
    return STAIRS_OK;
  }
  const int chunk = ctx->cfg.prefill_chunk > 0 ? ctx->cfg.prefill_chunk : 256;
  for (int c0 = 0; c0 < n_ctx; c0 += chunk) {
    const int n = std::min(chunk, n_ctx - c0);
    RowParams p = base_rows(ctx);
    p.mode = ROWS_PREFILL; p.slot = slot; p.first = c0; p.n_rows = n;
    int rc = launch_rows(ctx, p, n);
    if (rc) return rc;
    rc = forward(ctx, M, n, 0, 0, nullptr);
    if (rc) return rc;
  }
  return STAIRS_OK;
}

}  // namespace

// =============================================================================================
// C-ABI
// =============================================================================================
extern "C" {

size_t stairs_workspace_bytes(const stairs_config* cfg) {
  if (!cfg) return 0;
  Layout L{};
  const char* why = nullptr;
  if (!compute_layout(*cfg, &L, &why)) { g_init_error = why ? why : "bad configuration"; return 0; }
  return L.total;
}

int stairs_init(const stairs_config* cfg, const stairs_weights* target, const stairs_weights* draft, stairs_ctx** out) {
  if (!cfg || !target || !out) return fail(nullptr, STAIRS_EINVAL, "cfg, target and out must not be NULL");
  *out = nullptr;
  Layout L{};
  const char* why = nullptr;
  if (!compute_layout(*cfg, &L, &why)) return fail(nullptr, STAIRS_EINVAL, "%s", why ? why : "bad configuration");
  const bool has_draft = cfg->draft.n_layers > 0;
  if (has_draft && !draft) return fail(nullptr, STAIRS_EINVAL, "draft weights missing");
  if (!cfg->workspace || (reinterpret_cast<uintptr_t>(cfg->workspace) & 255))
    return fail(nullptr, STAIRS_EINVAL, "workspace must be a 256-byte aligned device pointer");
  if (cfg->workspace_bytes < L.total)
    return fail(nullptr, STAIRS_ENOSPC, "workspace too small: %zu < %zu bytes", cfg->workspace_bytes, L.total);
  auto check_w = [&](const stairs_model& m, const stairs_weights* w) -> const char* {
    if (!w->tok_emb || !w->final_norm_w || !w->lm_head || (m.n_layers > 0 && !w->layers)) return "global weight pointer missing";
    if (m.pos == 0 && !w->pos_emb) return "pos_emb missing";
    if (m.norm == 0 && !w->final_norm_b) return "final_norm_b missing";
    for (int l = 0; l < m.n_layers; ++l) {
      const stairs_layer_w& y = w->layers[l];
      if (!y.norm1_w || !y.wq || !y.wk || !y.wv || !y.wo || !y.norm2_w || !y.w_gate_or_fc1 || !y.w_down_or_fc2)
        return "layer weight pointer missing";
      if (m.act == 1 && !y.w_up) return "w_up missing for SwiGLU";
      if (m.norm == 0 && (!y.norm1_b || !y.norm2_b)) return "LayerNorm bias missing";
    }
    return nullptr;
  };
  if ((why = check_w(cfg->target, target))) return fail(nullptr, STAIRS_EINVAL, "target: %s", why);
  if (has_draft && (why = check_w(cfg->draft, draft))) return fail(nullptr, STAIRS_EINVAL, "draft: %s", why);

  cudaError_t e = cudaSetDevice(cfg->device);
  if (e != cudaSuccess) return fail(nullptr, STAIRS_ECUDA, "cudaSetDevice(%d): %s", cfg->device, cudaGetErrorString(e));
  stairs_ctx* ctx = new (std::nothrow) stairs_ctx();
  if (!ctx) return fail(nullptr, STAIRS_ENOSPC, "out of host memory");
  ctx->cfg = *cfg;
  ctx->lay = L;
  ctx->stream = reinterpret_cast<cudaStream_t>(cfg->stream);
  ctx->ws = reinterpret_cast<char*>(cfg->workspace);
  auto fill = [&](DevModel& M, const stairs_model& m, const stairs_weights* w) {
    M.m = m; M.present = true; M.w = *w;
    M.layers.assign(w->layers, w->layers + m.n_layers);
    M.w.layers = M.layers.data();
  };
  fill(ctx->target, cfg->target, target);
  ctx->target.kpool = ctx->ws + L.kv_t_k; ctx->target.vpool = ctx->ws + L.kv_t_v; ctx->target.kv_layer_bytes = L.kv_t_layer;
  if (has_draft) {
    fill(ctx->draft, cfg->draft, draft);
    ctx->draft.kpool = ctx->ws + L.kv_d_k; ctx->draft.vpool = ctx->ws + L.kv_d_v; ctx->draft.kv_layer_bytes = L.kv_d_layer;
  }
  ctx->pages.resize(cfg->max_requests);
  ctx->n_seq_ub.assign(cfg->max_requests, 0);
  ctx->active.assign(cfg->max_requests, 0);
  for (int p = L.n_pages - 1; p >= 0; --p) ctx->free_pages.push_back(p);
  // clear status words, sequences, lengths and page tables; and the K/V pools: a position is always
  // written before it becomes visible, but the attention phases fetch whole page slices, whose
  // rows past a request's end are masked yet multiplied (by zero weights), so they must be finite
  e = cudaMemsetAsync(ctx->ws, 0, L.tok, ctx->stream);
  if (e == cudaSuccess && L.total > L.kv_t_k) e = cudaMemsetAsync(ctx->ws + L.kv_t_k, 0, L.total - L.kv_t_k, ctx->stream);
  if (e == cudaSuccess && L.kv_t_k > L.gemm_counters)  // split-tile counters start at zero and return to zero
    e = cudaMemsetAsync(ctx->ws + L.gemm_counters, 0, L.w13_t - L.gemm_counters, ctx->stream);
  if (e == cudaSuccess && L.mk_partial_bytes) e = cudaMemsetAsync(ctx->ws + L.mk_partial, 0xff, L.mk_partial_bytes, ctx->stream);   // all slots empty
  if (e == cudaSuccess && L.mk_partial_bytes) e = cudaMemsetAsync(ctx->ws + L.attn_part, 0xff, 2 * L.attn_part_bytes, ctx->stream);   // and all parked attention states
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
  if (e == cudaSuccess) e = cudaEventCreate(&ctx->call_begin);
  if (e == cudaSuccess) e = cudaEventCreate(&ctx->call_end);
  if (e != cudaSuccess) {
    int rc = fail(nullptr, STAIRS_ECUDA, "context set-up failed: %s", cudaGetErrorString(e));
    delete ctx;
    return rc;
  }
  // tensor-core path: bf16 weights on a device with tcgen05 (compute capability 10.x)
  {
    int major = 0;
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, cfg->device);
    cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, cfg->device);
    ctx->wait_limit = cfg->wait_limit_cycles ? cfg->wait_limit_cycles : 2000000000ull;
    e = cudaHostAlloc(reinterpret_cast<void**>(&ctx->status_host), STATUS_WORDS * 4, cudaHostAllocMapped);
    if (e == cudaSuccess) {
      memset(ctx->status_host, 0, STATUS_WORDS * 4);
      e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&ctx->status_dev), ctx->status_host, 0);
    }
    if (e == cudaSuccess) {
      const size_t nd = (size_t)cfg->max_requests * std::max(cfg->k_max, 1), ntt = (size_t)cfg->max_requests * (cfg->k_max + 1);
      ctx->io_draft = 0; ctx->io_tt = nd; ctx->io_al = nd + ntt;
      e = cudaHostAlloc(reinterpret_cast<void**>(&ctx->io_host), (nd + ntt + cfg->max_requests) * 4, cudaHostAllocMapped);
      if (e == cudaSuccess) e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&ctx->io_dev), ctx->io_host, 0);
    }
    if (e != cudaSuccess) {
      int rc = fail(nullptr, STAIRS_ECUDA, "pinned status / result block set-up failed: %s", cudaGetErrorString(e));
      if (ctx->status_host) cudaFreeHost(ctx->status_host);
      if (ctx->io_host) cudaFreeHost(ctx->io_host);
      delete ctx;
      return rc;
    }
    if (cfg->target.wdtype == 1 && cfg->gemm_impl != 1) {
      if (major != 10) {
        int rc = fail(nullptr, STAIRS_EUNSUPPORTED, "bf16 models need an sm_100 device (found compute capability %d.x)", major);
        stairs_destroy(ctx);
        return rc;
      }
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
      if (e != cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess) {
        int rc = fail(nullptr, STAIRS_ECUDA, "cuTensorMapEncodeTiled is not available from the driver");
        stairs_destroy(ctx);
        return rc;
      }
      ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
      e = cudaFuncSetAttribute(tc::k_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_LIMIT);
      int rc = e == cudaSuccess ? build_weight_maps(ctx, ctx->target) : fail(ctx, STAIRS_ECUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
      if (!rc && has_draft) rc = build_weight_maps(ctx, ctx->draft);
      if (rc) {
        g_init_error = ctx->err;
        stairs_destroy(ctx);
        return rc;
      }
      ctx->use_tc = true;
      // persistent whole-pass kernel (gemm_impl 0 only; 2 keeps one launch per GEMM)
      int coop = 0;
      cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, cfg->device);
      const int hdm = has_draft ? std::max(cfg->target.head_dim, cfg->draft.head_dim) : cfg->target.head_dim;
      const long long worst_chunks = ((long long)cfg->max_seq_len + mk::ATT_CHUNK - 1) / mk::ATT_CHUNK;
      const int hkvm = has_draft ? std::max(cfg->target.n_kv_heads, cfg->draft.n_kv_heads) : cfg->target.n_kv_heads;
      const bool fits = mk::pick_stages(MK_MAX_ROWS, hdm, 1, 1) >= 3 && worst_chunks * hkvm / 64 <= 2 * std::min(ctx->sm_count, TC_GRID_MAX);
      if (coop && fits && cfg->gemm_impl == 0) {
        e = cudaFuncSetAttribute(mk::k_forward, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_LIMIT);
        if (e == cudaSuccess) {
          ctx->use_mk = true;
          ctx->target.prog_base = ctx->ws + L.prog_t; ctx->target.prog_slot_bytes = L.prog_slot_t; ctx->target.prog_maps_off = L.prog_maps_off_t;
          ctx->draft.prog_base = ctx->ws + L.prog_d; ctx->draft.prog_slot_bytes = L.prog_slot_d; ctx->draft.prog_maps_off = L.prog_maps_off_d;
          int rc2 = setup_mk_model(ctx, ctx->target, L.rope_t, L.aux_t, L.w13_t, nullptr);
          if (!rc2 && has_draft) rc2 = setup_mk_model(ctx, ctx->draft, L.rope_d, L.aux_d, L.w13_d, &ctx->target);
          if (rc2) {
            g_init_error = ctx->err;
            stairs_destroy(ctx);
            return rc2;
          }
          // Early-exit assistant (its layers are the main model's first layers, same tensors): the K/V
          // it would compute for a position are bit for bit those the main model computes for the
          // same token (results do not depend on a call's row count), so it works on the main
          // model's pools: no second prefill, no second cache.  Every position it writes is one the
          // next validation pass writes again before reading it.
          if (has_draft && mk_eligible(ctx, ctx->draft, 1) && mk_eligible(ctx, ctx->target, 1) &&
              cfg->draft.n_layers <= cfg->target.n_layers && cfg->draft.n_heads == cfg->target.n_heads &&
              cfg->draft.n_kv_heads == cfg->target.n_kv_heads && cfg->draft.head_dim == cfg->target.head_dim &&
              cfg->draft.d_ff == cfg->target.d_ff) {
            bool same = true;
            for (int l = 0; l < cfg->draft.n_layers && same; ++l)
              same = memcmp(&ctx->draft.layers[l], &ctx->target.layers[l], sizeof(stairs_layer_w)) == 0;
            if (same) {
              ctx->draft_shares_kv = true;
              ctx->draft.kpool = ctx->target.kpool; ctx->draft.vpool = ctx->target.vpool;
              ctx->draft.kv_layer_bytes = ctx->target.kv_layer_bytes;
            }
          }
        }
      }
    }
  }
  *out = ctx;
  return STAIRS_OK;
}

int stairs_prefill(stairs_ctx* ctx, int req, const int32_t* prompt_host, int n_prompt) {
  int rc = check_slot(ctx, req, false);
  if (rc) return rc;
  if (!prompt_host || n_prompt < 2) return fail(ctx, STAIRS_EINVAL, "prompt must hold at least 2 tokens");
  if (n_prompt + 1 > ctx->cfg.max_seq_len)
    return fail(ctx, STAIRS_ENOSPC, "prompt of %d tokens does not fit max_seq_len %d", n_prompt, ctx->cfg.max_seq_len);
  for (int i = 0; i < n_prompt; ++i)
    if (prompt_host[i] < 0 || prompt_host[i] >= ctx->cfg.target.vocab)
      return fail(ctx, STAIRS_EINVAL, "prompt token %d out of range at %d", prompt_host[i], i);
  release_pages(ctx, req);
  rc = ensure_pages(ctx, req, n_prompt);
  if (rc) return rc;
  int* seq = reinterpret_cast<int*>(ctx->ws + ctx->lay.seq) + (size_t)req * ctx->cfg.max_seq_len;
  int* nseq = reinterpret_cast<int*>(ctx->ws + ctx->lay.n_seq) + req;
  CK(cudaMemcpyAsync(seq, prompt_host, (size_t)n_prompt * 4, cudaMemcpyHostToDevice, ctx->stream));
  CK(cudaMemcpyAsync(nseq, &n_prompt, 4, cudaMemcpyHostToDevice, ctx->stream));
  ctx->active[req] = 1;
  ctx->n_seq_ub[req] = n_prompt;
  rc = prefill_model(ctx, ctx->target, req, n_prompt - 1);
  if (rc) return rc;
  // (an assistant that shares the main model's cache finds the prompt's K/V of its layers there already)
  if (ctx->draft.present && !ctx->draft_shares_kv) rc = prefill_model(ctx, ctx->draft, req, n_prompt - 1);
  return rc;
}

int stairs_draft(stairs_ctx* ctx, int req, int k, int32_t* draft_dev) {
  int rc = check_slot(ctx, req, true);
  if (rc) return rc;
  if (!ctx->draft.present) return fail(ctx, STAIRS_ESTATE, "no draft model configured");
  if (k < 0 || k > ctx->cfg.k_max || (k > 0 && !draft_dev)) return fail(ctx, STAIRS_EINVAL, "draft length %d outside 0..k_max", k);
  if (k == 0) return STAIRS_OK;
  if (ctx->n_seq_ub[req] + k > ctx->cfg.max_seq_len)
    return fail(ctx, STAIRS_ENOSPC, "request %d: sequence would exceed max_seq_len", req);
  rc = ensure_pages(ctx, req, ctx->n_seq_ub[req] + k);
  if (rc) return rc;
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(ctx->ws + ctx->lay.keys);
  for (int j = 0; j < k; ++j) {
    RowParams p = base_rows(ctx);
    p.slot = req; p.draft = draft_dev; p.first = j;
    p.mode = j == 0 ? ROWS_DRAFT_FIRST : ROWS_DRAFT_NEXT;
    const int T = (j == 0 && !ctx->draft_shares_kv) ? 2 : 1;
    if (mk_eligible(ctx, ctx->draft, T)) {
      MkCall c;
      c.mode = j == 0 ? mk::CALL_DRAFT_FIRST : mk::CALL_DRAFT_NEXT;
      c.slot = req; c.draft_step = j; c.draft = draft_dev; c.draft_out = draft_dev;
      if ((rc = launch_forward_mk(ctx, ctx->draft, T, T - 1, 1, c))) return rc;
      continue;
    }
    if ((rc = launch_rows(ctx, p, T))) return rc;
    if ((rc = forward(ctx, ctx->draft, T, T - 1, 1, nullptr))) return rc;
    k_take_token<<<1, 32, 0, ctx->stream>>>(keys, T - 1, draft_dev, j);
    ctx->launches++;
  }
  CK(cudaGetLastError());
  return STAIRS_OK;
}

int stairs_validate(stairs_ctx* ctx, int n_req, const int32_t* req_ids_host, const int32_t* k_host,
                    const int32_t* draft_dev, int32_t* target_tokens_dev, int32_t* accept_len_dev,
                    float* logits_dev_or_null, int commit) {
  if (!ctx) return STAIRS_EINVAL;
  if (n_req <= 0 || n_req > ctx->cfg.max_requests || !req_ids_host || !k_host || !target_tokens_dev || !accept_len_dev)
    return fail(ctx, STAIRS_EINVAL, "bad validate arguments");
  std::vector<int> off(n_req);
  int T = 0;
  for (int i = 0; i < n_req; ++i) {
    int rc = check_slot(ctx, req_ids_host[i], true);
    if (rc) return rc;
    for (int j = 0; j < i; ++j)
      if (req_ids_host[j] == req_ids_host[i]) return fail(ctx, STAIRS_EINVAL, "request %d listed twice", req_ids_host[i]);
    if (k_host[i] < 0 || k_host[i] > ctx->cfg.k_max) return fail(ctx, STAIRS_EINVAL, "k[%d]=%d outside 0..k_max", i, k_host[i]);
    if (k_host[i] > 0 && !draft_dev) return fail(ctx, STAIRS_EINVAL, "draft_dev is NULL");
    off[i] = T;
    T += k_host[i] + 1;
  }
  for (int i = 0; i < n_req; ++i) {
    const int slot = req_ids_host[i];
    const int need = ctx->n_seq_ub[slot] + k_host[i] + 1;  // sequence length after a full accept
    if (need > ctx->cfg.max_seq_len) return fail(ctx, STAIRS_ENOSPC, "request %d: sequence would exceed max_seq_len", slot);
    int rc = ensure_pages(ctx, slot, need);
    if (rc) return rc;
  }
  char* ws = ctx->ws;
  const Layout& L = ctx->lay;
  if (ctx->profile) { ctx->ev_used = 0; cudaEventRecord(ctx->call_begin, ctx->stream); }
  if (mk_eligible(ctx, ctx->target, T)) {
    MkCall c;
    c.mode = mk::CALL_VALIDATE; c.n_req = n_req; c.draft = draft_dev;
    c.req_host = req_ids_host; c.k_host = k_host; c.off_host = off.data();
    c.target_tokens = target_tokens_dev; c.accept_len = accept_len_dev; c.commit = commit; c.logits = logits_dev_or_null;
    int rc = launch_forward_mk(ctx, ctx->target, T, 0, T, c);
    if (rc) return rc;
    if (ctx->profile) cudaEventRecord(ctx->call_end, ctx->stream);
    if (commit)
      for (int i = 0; i < n_req; ++i) ctx->n_seq_ub[req_ids_host[i]] += k_host[i] + 1;
    return STAIRS_OK;
  }
  CK(cudaMemcpyAsync(ws + L.val_req, req_ids_host, (size_t)n_req * 4, cudaMemcpyHostToDevice, ctx->stream));
  CK(cudaMemcpyAsync(ws + L.val_k, k_host, (size_t)n_req * 4, cudaMemcpyHostToDevice, ctx->stream));
  CK(cudaMemcpyAsync(ws + L.val_off, off.data(), (size_t)n_req * 4, cudaMemcpyHostToDevice, ctx->stream));
  ctx->in_validate = true;
  RowParams p = base_rows(ctx);
  p.mode = ROWS_VALIDATE; p.n_req = n_req; p.draft = draft_dev;
  int rc = launch_rows(ctx, p, n_req * (ctx->cfg.k_max + 1));
  if (!rc) rc = forward(ctx, ctx->target, T, 0, T, logits_dev_or_null);
  ctx->in_validate = false;
  if (rc) return rc;
  AcceptParams a{};
  a.n_req = n_req; a.val_req = p.val_req; a.val_k = p.val_k; a.val_off = p.val_off;
  a.draft = draft_dev; a.k_max = ctx->cfg.k_max;
  a.keys = reinterpret_cast<unsigned long long*>(ws + L.keys);
  a.target_tokens = target_tokens_dev; a.accept_len = accept_len_dev; a.commit = commit;
  a.seq = reinterpret_cast<int*>(ws + L.seq); a.n_seq = reinterpret_cast<int*>(ws + L.n_seq);
  a.max_seq_len = ctx->cfg.max_seq_len;
  k_accept<<<(n_req + 63) / 64, 64, 0, ctx->stream>>>(a);
  ctx->launches++;
  CK(cudaGetLastError());
  if (ctx->profile) cudaEventRecord(ctx->call_end, ctx->stream);
  if (commit)
    for (int i = 0; i < n_req; ++i) ctx->n_seq_ub[req_ids_host[i]] += k_host[i] + 1;
  return STAIRS_OK;
}

int stairs_validate_host(stairs_ctx* ctx, int n_req, const int32_t* req_ids_host, const int32_t* k_host,
                         const int32_t* draft_host, int32_t* target_tokens_host, int32_t* accept_len_host, int commit) {
  if (!ctx) return STAIRS_EINVAL;
  if (n_req <= 0 || n_req > ctx->cfg.max_requests || !target_tokens_host || !accept_len_host)
    return fail(ctx, STAIRS_EINVAL, "bad validate arguments");
  char* ws = ctx->ws;
  const Layout& L = ctx->lay;
  const int km = ctx->cfg.k_max;
  int* d_dev = reinterpret_cast<int*>(ws + L.draft_buf);
  // drafts: staged in pinned memory, one asynchronous copy; results: the pass writes them straight
  // into pinned host memory, so nothing is copied back
  if (km > 0 && draft_host) {
    memcpy(ctx->io_host + ctx->io_draft, draft_host, (size_t)n_req * km * 4);
    CK(cudaMemcpyAsync(d_dev, ctx->io_host + ctx->io_draft, (size_t)n_req * km * 4, cudaMemcpyHostToDevice, ctx->stream));
  }
  int rc = stairs_validate(ctx, n_req, req_ids_host, k_host, draft_host ? d_dev : nullptr, ctx->io_dev + ctx->io_tt,
                           ctx->io_dev + ctx->io_al, nullptr, commit);
  if (rc) return rc;
  rc = stairs_sync(ctx);
  if (rc) return rc;
  memcpy(target_tokens_host, ctx->io_host + ctx->io_tt, (size_t)n_req * (km + 1) * 4);
  memcpy(accept_len_host, ctx->io_host + ctx->io_al, (size_t)n_req * 4);
  if (commit)  // the host now knows the exact new lengths
    for (int i = 0; i < n_req; ++i) ctx->n_seq_ub[req_ids_host[i]] += accept_len_host[i] - k_host[i];
  return STAIRS_OK;
}

}  // extern "C"

namespace {

// The generation loop behind stairs_generate and stairs_generate_adaptive.  adaptive: the draft
// length follows the acceptance (all drafts kept: two more next time, otherwise one fewer, never
// below one), the schedule of the sequential assisted generation the paper compares with.
int generate_loop(stairs_ctx* ctx, int req, const int32_t* prompt_host, int n_prompt, int k, int max_new,
                  int32_t eos, int32_t* out_host, int32_t* n_out, stairs_stats* stats, bool adaptive) {
  int rc = check_slot(ctx, req, false);
  if (rc) return rc;
  if (!out_host || !n_out || max_new < 0) return fail(ctx, STAIRS_EINVAL, "bad generate arguments");
  if (k < 0 || k > ctx->cfg.k_max) return fail(ctx, STAIRS_EINVAL, "k=%d outside 0..k_max", k);
  if (k > 0 && !ctx->draft.present) return fail(ctx, STAIRS_ESTATE, "k > 0 needs a draft model");
  if (n_prompt + max_new > ctx->cfg.max_seq_len) return fail(ctx, STAIRS_ENOSPC, "prompt + max_new exceeds max_seq_len");
  stairs_stats s{};
  cudaEvent_t e0, e1, e2, e3;
  CK(cudaEventCreate(&e0)); CK(cudaEventCreate(&e1)); CK(cudaEventCreate(&e2)); CK(cudaEventCreate(&e3));
  auto cleanup = [&]() { cudaEventDestroy(e0); cudaEventDestroy(e1); cudaEventDestroy(e2); cudaEventDestroy(e3); };
  float ms = 0.f;
  {
    cudaError_t pe = cudaEventRecord(e0, ctx->stream);
    rc = pe == cudaSuccess ? stairs_prefill(ctx, req, prompt_host, n_prompt) : fail(ctx, STAIRS_ECUDA, "cudaEventRecord: %s", cudaGetErrorString(pe));
    if (!rc && (pe = cudaEventRecord(e1, ctx->stream)) != cudaSuccess) rc = fail(ctx, STAIRS_ECUDA, "cudaEventRecord: %s", cudaGetErrorString(pe));
    if (!rc) rc = stairs_sync(ctx);
    if (!rc && (pe = cudaEventElapsedTime(&ms, e0, e1)) != cudaSuccess) rc = fail(ctx, STAIRS_ECUDA, "cudaEventElapsedTime: %s", cudaGetErrorString(pe));
    if (rc) { cleanup(); return rc; }
  }
  s.prefill_ms = ms;
  const int km = ctx->cfg.k_max;
  int* d_dev = reinterpret_cast<int*>(ctx->ws + ctx->lay.draft_buf);
  // results land in pinned host memory (written by the pass itself); the drafted tokens come back
  // with one small copy into the same block
  int* tt_dev = ctx->io_dev + ctx->io_tt;
  int* al_dev = ctx->io_dev + ctx->io_al;
  const int* tt = ctx->io_host + ctx->io_tt;
  const int* al_h = ctx->io_host + ctx->io_al;
  int* draft_h = ctx->io_host + ctx->io_draft;
  (void)km;
  int produced = 0;
  bool stop = false;
  cudaError_t ce = cudaSuccess;
  int k_cur = k;
  while (produced < max_new && !stop) {
    const int k_eff = std::min(k_cur, max_new - produced - 1);
    if ((ce = cudaEventRecord(e1, ctx->stream)) != cudaSuccess) break;
    if (k_eff > 0 && (rc = stairs_draft(ctx, req, k_eff, d_dev))) break;
    if ((ce = cudaEventRecord(e2, ctx->stream)) != cudaSuccess) break;
    if ((rc = stairs_validate(ctx, 1, &req, &k_eff, d_dev, tt_dev, al_dev, nullptr, 1))) break;
    if ((ce = cudaEventRecord(e3, ctx->stream)) != cudaSuccess) break;
    if (k_eff > 0 && (ce = cudaMemcpyAsync(draft_h, d_dev, (size_t)k_eff * 4, cudaMemcpyDeviceToHost, ctx->stream)) != cudaSuccess) break;
    if ((rc = stairs_sync(ctx))) break;
    const int al = al_h[0];
    ctx->n_seq_ub[req] += al - k_eff;
    if ((ce = cudaEventElapsedTime(&ms, e1, e2)) != cudaSuccess) break;
    s.draft_ms += ms;
    if ((ce = cudaEventElapsedTime(&ms, e2, e3)) != cudaSuccess) break;
    s.validate_ms += ms;
    s.iterations++; s.drafted += k_eff; s.accepted += al;
    if (adaptive && k_eff > 0) k_cur = al == k_eff ? std::min(k_cur + 2, ctx->cfg.k_max) : std::max(1, k_cur - 1);
    for (int r = 0; r <= al && !stop; ++r) {
      const int t = r < al ? draft_h[r] : tt[al];
      if (produced < max_new) out_host[produced] = t;
      produced++; s.emitted++;
      if (eos >= 0 && t == eos) stop = true;
    }
  }
  if (!rc && ce != cudaSuccess) rc = fail(ctx, STAIRS_ECUDA, "stairs_generate: %s", cudaGetErrorString(ce));
  if (!rc) {
    cudaError_t fe = cudaEventRecord(e3, ctx->stream);
    rc = fe == cudaSuccess ? stairs_sync(ctx) : fail(ctx, STAIRS_ECUDA, "cudaEventRecord: %s", cudaGetErrorString(fe));
    if (!rc && (fe = cudaEventElapsedTime(&ms, e0, e3)) != cudaSuccess) rc = fail(ctx, STAIRS_ECUDA, "cudaEventElapsedTime: %s", cudaGetErrorString(fe));
    s.total_ms = ms;
  }
  cleanup();
  if (rc) return rc;
  *n_out = std::min(produced, max_new);
  if (stats) *stats = s;
  return STAIRS_OK;
}

}  // namespace

extern "C" {

int stairs_generate(stairs_ctx* ctx, int req, const int32_t* prompt_host, int n_prompt, int k, int max_new,
                    int32_t eos, int32_t* out_host, int32_t* n_out, stairs_stats* stats) {
  return generate_loop(ctx, req, prompt_host, n_prompt, k, max_new, eos, out_host, n_out, stats, false);
}

int stairs_generate_adaptive(stairs_ctx* ctx, int req, const int32_t* prompt_host, int n_prompt, int k_first, int max_new,
                             int32_t eos, int32_t* out_host, int32_t* n_out, stairs_stats* stats) {
  if (ctx && k_first < 1) return fail(ctx, STAIRS_EINVAL, "k_first=%d: the adaptive schedule starts from at least one drafted token", k_first);
  return generate_loop(ctx, req, prompt_host, n_prompt, k_first, max_new, eos, out_host, n_out, stats, true);
}

int stairs_sequence(stairs_ctx* ctx, int req, int32_t* seq_host, int capacity, int32_t* n_seq) {
  int rc = check_slot(ctx, req, true);
  if (rc) return rc;
  if (!n_seq) return fail(ctx, STAIRS_EINVAL, "n_seq is NULL");
  int n = 0;
  CK(cudaMemcpyAsync(&n, reinterpret_cast<int*>(ctx->ws + ctx->lay.n_seq) + req, 4, cudaMemcpyDeviceToHost, ctx->stream));
  if ((rc = stairs_sync(ctx))) return rc;
  *n_seq = n;
  ctx->n_seq_ub[req] = n;
  if (seq_host && capacity > 0) {
    const int* seq = reinterpret_cast<int*>(ctx->ws + ctx->lay.seq) + (size_t)req * ctx->cfg.max_seq_len;
    CK(cudaMemcpyAsync(seq_host, seq, (size_t)std::min(n, capacity) * 4, cudaMemcpyDeviceToHost, ctx->stream));
    rc = stairs_sync(ctx);
  }
  return rc;
}

int stairs_truncate(stairs_ctx* ctx, int req, int n_tokens) {
  int rc = check_slot(ctx, req, true);
  if (rc) return rc;
  if (n_tokens < 2 || n_tokens > ctx->n_seq_ub[req]) return fail(ctx, STAIRS_EINVAL, "truncate length %d outside 2..%d", n_tokens, ctx->n_seq_ub[req]);
  CK(cudaMemcpyAsync(reinterpret_cast<int*>(ctx->ws + ctx->lay.n_seq) + req, &n_tokens, 4, cudaMemcpyHostToDevice, ctx->stream));
  ctx->n_seq_ub[req] = n_tokens;
  return STAIRS_OK;
}

int stairs_sync(stairs_ctx* ctx) {
  if (!ctx) return STAIRS_EINVAL;
  CK(cudaStreamSynchronize(ctx->stream));
  if (ctx->status_host && ctx->status_host[STATUS_ERROR]) {
    const unsigned int code = ctx->status_host[STATUS_ERROR];
    const unsigned int where[5] = {ctx->status_host[STATUS_WHERE], ctx->status_host[2], ctx->status_host[3], ctx->status_host[4],
                                   ctx->status_host[5]};
    ctx->status_host[STATUS_ERROR] = 0;
    for (int i = 1; i <= 5; ++i) ctx->status_host[i] = 0;
    cudaMemsetAsync(ctx->ws + ctx->lay.mk_bar, 0, 64, ctx->stream);   // barrier count and abort word
    cudaMemsetAsync(ctx->ws + ctx->lay.gemm_counters, 0, (size_t)TC_COUNTERS * 4, ctx->stream);
    if (ctx->lay.mk_partial_bytes) cudaMemsetAsync(ctx->ws + ctx->lay.mk_partial, 0xff, ctx->lay.mk_partial_bytes, ctx->stream);   // all partial-sum slots empty again
    if (ctx->lay.mk_partial_bytes) cudaMemsetAsync(ctx->ws + ctx->lay.attn_part, 0xff, 2 * ctx->lay.attn_part_bytes, ctx->stream);
    cudaStreamSynchronize(ctx->stream);
    ctx->bar_base = 0;
    // kind: 1 shared-memory barrier (block, thread, parity), 2 grid barrier (block, thread, target),
    // 3 split-tile partial sums (phase, block, last block of the tile, tile)
    // 4 attention-scratch guard (unit slot, slots available, request, unit), 5 parked attention states (phase, block)
    return fail(ctx, (int)code, "%s (code %u; first: kind %u at %u, %u, %u, %u); results of the last calls are invalid",
                where[0] == 4u ? "the device-side attention scratch was too small for a call" : "a device-side bounded wait expired",
                code, where[0], where[1], where[2], where[3], where[4]);
  }
  return STAIRS_OK;
}

int64_t stairs_launch_count(const stairs_ctx* ctx) { return ctx ? ctx->launches : 0; }

int stairs_profile(stairs_ctx* ctx, int enable) {
  if (!ctx) return STAIRS_EINVAL;
  if (enable && ctx->ev.empty()) {
    ctx->ev.resize(4096);
    for (auto& e : ctx->ev) CK(cudaEventCreate(&e));
  }
  ctx->profile = enable != 0;
  ctx->ev_used = 0;
  return STAIRS_OK;
}

int stairs_profile_read(stairs_ctx* ctx, float* gemm_ms, int32_t* gemm_launches, float* call_ms) {
  if (!ctx) return STAIRS_EINVAL;
  if (!ctx->profile) return fail(ctx, STAIRS_ESTATE, "profiling is off");
  int rc = stairs_sync(ctx);
  if (rc) return rc;
  float total = 0.f;
  for (int i = 0; i + 1 < ctx->ev_used; i += 2) {
    float ms = 0.f;
    CK(cudaEventElapsedTime(&ms, ctx->ev[i], ctx->ev[i + 1]));
    total += ms;
  }
  if (gemm_ms) *gemm_ms = total;
  if (gemm_launches) *gemm_launches = ctx->ev_used / 2;
  if (call_ms) { float ms = 0.f; CK(cudaEventElapsedTime(&ms, ctx->call_begin, ctx->call_end)); *call_ms = ms; }
  return STAIRS_OK;
}

int stairs_debug_buffer(stairs_ctx* ctx, int which, void** ptr_dev, size_t* bytes) {
  if (!ctx || !ptr_dev || !bytes) return STAIRS_EINVAL;
  const Layout& L = ctx->lay;
  const size_t off[7] = {L.x, L.h, L.qkv, L.q, L.o, L.ff, L.logits};
  const size_t keys_end = L.x;
  switch (which) {
    case 0: *ptr_dev = ctx->ws + off[0]; *bytes = off[1] - off[0]; break;
    case 1: *ptr_dev = ctx->ws + off[1]; *bytes = off[2] - off[1]; break;
    case 2: *ptr_dev = ctx->ws + off[2]; *bytes = off[3] - off[2]; break;
    case 3: *ptr_dev = ctx->ws + off[4]; *bytes = off[5] - off[4]; break;
    case 4: *ptr_dev = ctx->ws + off[5]; *bytes = off[6] - off[5]; break;
    case 5: *ptr_dev = ctx->ws + L.keys; *bytes = keys_end - L.keys; break;
    case 6: *ptr_dev = ctx->ws + L.mk_trace; *bytes = L.mk_stats - L.mk_trace; break;
    case 7: *ptr_dev = ctx->ws + L.mk_partial; *bytes = L.mk_partial_bytes; break;
    case 8: *ptr_dev = ctx->ws + L.attn_part; *bytes = L.mk_partial_bytes ? 2 * L.attn_part_bytes : 0; break;
    default: return fail(ctx, STAIRS_EINVAL, "unknown buffer %d", which);
  }
  return STAIRS_OK;
}

int stairs_debug_tune(stairs_ctx* ctx, int what, long long value) {
  if (!ctx) return STAIRS_EINVAL;
  switch (what) {
    case 0:
      if (value != 0 && value != 1 && value != 2) return fail(ctx, STAIRS_EINVAL, "k-blocks per stage must be 0 (auto), 1 or 2");
      ctx->kps_force = (int)value;
      break;
    case 1:
      if (value < 0 || value > mk::MAX_KV_BUF) return fail(ctx, STAIRS_EINVAL, "K/V chunk buffers must be 0 (auto) .. %d", mk::MAX_KV_BUF);
      ctx->att_nbuf_force = (int)value;
      break;
    case 2: ctx->att_tma_off = value ? 1 : 0; break;
    case 3: ctx->att_tc_off = value == 1 ? 1 : 0; ctx->att_tc_force = value == 2 ? 1 : 0; break;
    default: return fail(ctx, STAIRS_EINVAL, "unknown tuning knob %d", what);
  }
  // programs carry the tensor maps' box depth, which follows from the shared-memory plan
  for (bool& b : ctx->target.prog_built) b = false;
  for (bool& b : ctx->draft.prog_built) b = false;
  return STAIRS_OK;
}

int stairs_reset(stairs_ctx* ctx, int req) {
  int rc = check_slot(ctx, req, false);
  if (rc) return rc;
  release_pages(ctx, req);
  int zero = 0;
  CK(cudaMemcpyAsync(reinterpret_cast<int*>(ctx->ws + ctx->lay.n_seq) + req, &zero, 4, cudaMemcpyHostToDevice, ctx->stream));
  return STAIRS_OK;
}

int stairs_destroy(stairs_ctx* ctx) {
  if (!ctx) return STAIRS_EINVAL;
  cudaStreamSynchronize(ctx->stream);
  for (auto& e : ctx->ev) cudaEventDestroy(e);
  if (ctx->call_begin) cudaEventDestroy(ctx->call_begin);
  if (ctx->call_end) cudaEventDestroy(ctx->call_end);
  if (ctx->status_host) cudaFreeHost(ctx->status_host);
  if (ctx->io_host) cudaFreeHost(ctx->io_host);
  delete ctx;
  return STAIRS_OK;
}

const char* stairs_last_error(const stairs_ctx* ctx) { return ctx ? ctx->err.c_str() : g_init_error.c_str(); }

}  // extern "C"

// =============================================================================================
// Allocation-free argmax + accept on caller-provided logits (see stairs_accept_static in the
// header).  The only scratch, one packed argmax key per row, is this fixed device array; the
// host side must not use the symbol itself as a pointer, so its device address is looked up
// once per device with cudaGetSymbolAddress.
// =============================================================================================
namespace {

static __device__ __align__(256) unsigned long long g_static_keys[STAIRS_STATIC_MAX_ROWS];

struct StaticAcceptParams {
  int n_req, k_max;
  int k[STAIRS_STATIC_MAX_REQ];
  int off[STAIRS_STATIC_MAX_REQ];
  const int* draft;
  int* target_tokens;
  int* accept_len;
};

// Same walk as k_accept without the commit step; reads the keys from the fixed array directly.
__global__ void k_accept_static(const __grid_constant__ StaticAcceptParams p) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= p.n_req) return;
  const int k = p.k[i], off = p.off[i];
  int a = -1;
  for (int r = 0; r <= k; ++r) {
    const int tr = argmax_key_index(g_static_keys[off + r]);
    p.target_tokens[i * (p.k_max + 1) + r] = tr;
    if (a < 0 && r < k && p.draft[i * p.k_max + r] != tr) a = r;
  }
  p.accept_len[i] = a < 0 ? k : a;
}

constexpr int kMaxDevices = 64;
unsigned long long* g_static_keys_addr[kMaxDevices] = {};

}  // namespace

extern "C" int stairs_accept_static(const float* logits_dev, int vocab, int ld, int n_req, const int32_t* k_host,
                                    const int32_t* draft_dev, int k_max, int32_t* target_tokens_dev,
                                    int32_t* accept_len_dev, void* stream) {
  stairs_ctx* ctx = nullptr;  // errors go to the thread-local text read by stairs_last_error(NULL)
  if (!logits_dev || !k_host || !target_tokens_dev || !accept_len_dev || vocab <= 0 || ld < vocab)
    return fail(nullptr, STAIRS_EINVAL, "stairs_accept_static: NULL buffer, vocab <= 0 or ld < vocab");
  if (n_req < 1 || n_req > STAIRS_STATIC_MAX_REQ)
    return fail(nullptr, STAIRS_ENOSPC, "stairs_accept_static: n_req=%d outside 1..%d", n_req, STAIRS_STATIC_MAX_REQ);
  if (k_max < 0 || k_max > 63) return fail(nullptr, STAIRS_EINVAL, "stairs_accept_static: k_max=%d outside 0..63", k_max);
  StaticAcceptParams p{};
  int rows = 0;
  for (int i = 0; i < n_req; ++i) {
    if (k_host[i] < 0 || k_host[i] > k_max)
      return fail(nullptr, STAIRS_EINVAL, "stairs_accept_static: k[%d]=%d outside 0..k_max=%d", i, k_host[i], k_max);
    if (k_host[i] > 0 && !draft_dev) return fail(nullptr, STAIRS_EINVAL, "stairs_accept_static: draft_dev is NULL");
    p.k[i] = k_host[i];
    p.off[i] = rows;
    rows += k_host[i] + 1;
  }
  if (rows > STAIRS_STATIC_MAX_ROWS)
    return fail(nullptr, STAIRS_ENOSPC, "stairs_accept_static: %d rows exceed the fixed scratch of %d rows", rows,
                STAIRS_STATIC_MAX_ROWS);
  int dev = 0;
  CK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return fail(nullptr, STAIRS_EUNSUPPORTED, "stairs_accept_static: device ordinal %d", dev);
  if (!g_static_keys_addr[dev]) {  // once per device, with that device current
    unsigned long long* ptr = nullptr;
    CK(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_keys));
    g_static_keys_addr[dev] = ptr;
  }
  unsigned long long* keys = g_static_keys_addr[dev];
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  // the array still holds the previous call's keys: the atomic max below needs zeros
  CK(cudaMemsetAsync(keys, 0, (size_t)rows * sizeof(unsigned long long), st));
  const int slices = std::max(1, std::min(64, vocab / 2048));
  k_argmax<<<dim3(slices, rows), 256, 0, st>>>(logits_dev, vocab, ld, keys);
  p.n_req = n_req; p.k_max = k_max; p.draft = draft_dev;
  p.target_tokens = target_tokens_dev; p.accept_len = accept_len_dev;
  k_accept_static<<<(n_req + 63) / 64, 64, 0, st>>>(p);
  CK(cudaGetLastError());
  return STAIRS_OK;
}
