// Row construction, embedding, norms, rotary + KV append, the plain attention kernel,
// vocabulary argmax and the accept/commit step.
//
// Row layout of one forward pass: T rows; row t carries a token id, an absolute position
// and the request slot whose KV pages it reads and writes.  Row t sees cache positions
// 0..pos[t] of its slot: for the stair rows of one request (consecutive positions) this is
// exactly the staircase mask - the shared prefix plus one more new position per row.
#pragma once
#include "common.cuh"

namespace stairs {

enum RowMode { ROWS_VALIDATE = 0, ROWS_PREFILL = 1, ROWS_DRAFT_FIRST = 2, ROWS_DRAFT_NEXT = 3 };

struct RowParams {
  int mode;
  int n_req;             // ROWS_VALIDATE: requests in this call
  const int* val_req;    // [n_req] slot ids
  const int* val_k;      // [n_req] draft lengths
  const int* val_off;    // [n_req] first row of each request
  const int* draft;      // ROWS_VALIDATE: [n_req, k_max]; ROWS_DRAFT_NEXT: the draft buffer
  int k_max;
  int slot;              // single-request modes
  int first;             // ROWS_PREFILL: first position of the chunk; ROWS_DRAFT_NEXT: step j
  int n_rows;            // ROWS_PREFILL: rows in the chunk
  const int* seq;        // [max_requests, max_seq_len]
  const int* n_seq;      // [max_requests]
  int max_seq_len;
  int vocab;
  int* tok; int* pos; int* req;            // outputs [T]
  unsigned long long* keys; int n_keys;    // argmax keys to clear
};

// Stair-row construction (paper Section 3.3, Fig. 4): request i contributes rows r = 0..k_i;
// row r ends with the last committed token (r = 0) or drafted token r-1, at position
// n_seq-1+r.  The other modes build the rows of a prefill chunk or of an assistant step.
__global__ void k_rows(RowParams p) {
  const int tid = blockIdx.x * blockDim.x + threadIdx.x;
  if (tid < p.n_keys) p.keys[tid] = 0ull;
  auto clampv = [&](int t) { return t < 0 ? 0 : (t >= p.vocab ? p.vocab - 1 : t); };
  if (p.mode == ROWS_VALIDATE) {
    // one thread per (request, row)
    const int i = tid / (p.k_max + 1), r = tid % (p.k_max + 1);
    if (i < p.n_req && r <= p.val_k[i]) {
      const int slot = p.val_req[i];
      const int P = p.n_seq[slot] - 1;
      const int t = p.val_off[i] + r;
      const int token = (r == 0) ? p.seq[(size_t)slot * p.max_seq_len + P] : p.draft[i * p.k_max + r - 1];
      p.tok[t] = clampv(token); p.pos[t] = P + r; p.req[t] = slot;
    }
  } else if (p.mode == ROWS_PREFILL) {
    if (tid < p.n_rows) {
      p.tok[tid] = clampv(p.seq[(size_t)p.slot * p.max_seq_len + p.first + tid]);
      p.pos[tid] = p.first + tid; p.req[tid] = p.slot;
    }
  } else if (p.mode == ROWS_DRAFT_FIRST) {
    // the assistant re-reads the last two committed tokens: after a fully accepted draft it
    // has not yet consumed the last drafted token; otherwise the first row recomputes a
    // cache entry that is already there, with identical values
    if (tid < 2) {
      const int n = p.n_seq[p.slot];
      p.tok[tid] = clampv(p.seq[(size_t)p.slot * p.max_seq_len + n - 2 + tid]);
      p.pos[tid] = n - 2 + tid; p.req[tid] = p.slot;
    }
  } else {
    if (tid == 0) {
      const int n = p.n_seq[p.slot];
      p.tok[0] = clampv(p.draft[p.first - 1]); p.pos[0] = n - 1 + p.first; p.req[0] = p.slot;
    }
  }
}

// x[t,:] = E[tok[t],:] (+ Epos[pos[t],:])
template <typename WT>
__global__ void k_embed(const WT* __restrict__ tok_emb, const WT* __restrict__ pos_emb,
                        const int* __restrict__ tok, const int* __restrict__ pos,
                        float* __restrict__ x, int d) {
  const int t = blockIdx.x;
  const WT* e = tok_emb + (size_t)tok[t] * d;
  const WT* pe = pos_emb ? pos_emb + (size_t)pos[t] * d : nullptr;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v = to_f32(e[i]);
    if (pe) v += to_f32(pe[i]);
    x[(size_t)t * d + i] = v;
  }
}

// h[t,:] = norm(x[t,:]) rounded to the GEMM operand type.  kind 0: LayerNorm (two-pass mean
// and variance), kind 1: RMSNorm.  One block per row.
template <typename AT>
__global__ void k_norm(const float* __restrict__ x, const float* __restrict__ g,
                       const float* __restrict__ b, AT* __restrict__ h, int d, int kind, float eps) {
  __shared__ float red[32];
  const int t = blockIdx.x;
  const float* xr = x + (size_t)t * d;
  float mean = 0.f;
  if (kind == 0) {
    float s = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) s += xr[i];
    mean = block_sum(s, red) / (float)d;
  }
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) { float c = xr[i] - mean; ss += c * c; }
  const float var = block_sum(ss, red) / (float)d;
  const float rstd = 1.0f / sqrtf(var + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v = (xr[i] - mean) * rstd * g[i];
    if (b) v += b[i];
    h[(size_t)t * d + i] = from_f32<AT>(v);
  }
}

// Rotary embedding of q and k, q to the attention operand buffer, k and v of the T new
// positions into the slot's pages.  qkv is fp32 [T, (Hq+2Hkv)*hd].  Element i of a head
// pairs with i + hd/2; angle = pos * theta^(-2i/hd).
template <typename AT, typename KT>
__global__ void k_rope_append(const float* __restrict__ qkv, const int* __restrict__ pos,
                              const int* __restrict__ req, const int* __restrict__ page_table,
                              AT* __restrict__ q_out, KT* __restrict__ kc, KT* __restrict__ vc,
                              int Hq, int Hkv, int hd, int rope, float theta,
                              int page_tokens, int max_pages) {
  const int t = blockIdx.x;
  const int p = pos[t];
  const int page = page_table[(size_t)req[t] * max_pages + p / page_tokens];
  const size_t slot = (size_t)page * page_tokens + (p % page_tokens);
  const int nq = Hq * hd, nkv = Hkv * hd, half = hd / 2;
  const float* row = qkv + (size_t)t * (nq + 2 * nkv);
  // q and k heads: (Hq + Hkv) * half rotation pairs
  for (int idx = threadIdx.x; idx < (Hq + Hkv) * half; idx += blockDim.x) {
    const int head = idx / half, i = idx % half;
    const float* src = row + (size_t)head * hd;  // k heads follow the q heads contiguously
    float a = src[i], b2 = src[i + half];
    if (rope) {
      const float inv = (float)exp2(-(double)(2 * i) / (double)hd * log2((double)theta));
      const float ang = (float)p * inv;
      float s, c;
      sincosf(ang, &s, &c);
      const float ra = a * c - b2 * s, rb = b2 * c + a * s;
      a = ra; b2 = rb;
    }
    if (head < Hq) {
      AT* dst = q_out + (size_t)t * nq + (size_t)head * hd;
      dst[i] = from_f32<AT>(a); dst[i + half] = from_f32<AT>(b2);
    } else {
      KT* dst = kc + slot * nkv + (size_t)(head - Hq) * hd;
      dst[i] = from_f32<KT>(a); dst[i + half] = from_f32<KT>(b2);
    }
  }
  const float* vsrc = row + nq + nkv;
  for (int i = threadIdx.x; i < nkv; i += blockDim.x) vc[slot * nkv + i] = from_f32<KT>(vsrc[i]);
}

// Plain attention over the paged cache: one block per (query head, row), four warps; the
// chunk of 32 positions starting at 32*c belongs to warp c % 4, whatever the batch, so a
// row's result does not depend on which other rows are in the call.  Within a chunk each
// lane scores one position; the four partial softmax states are merged in a fixed order.
template <typename AT, typename KT, int MAXD>
__global__ void __launch_bounds__(128)
k_attn_plain(const AT* __restrict__ q, const KT* __restrict__ kc, const KT* __restrict__ vc,
             const int* __restrict__ page_table, const int* __restrict__ req,
             const int* __restrict__ pos, AT* __restrict__ o, int Hq, int Hkv, int hd,
             int page_tokens, int max_pages, float scale) {
  extern __shared__ float sm[];
  float* qs = sm;                 // [hd]
  float* accs = sm + hd;          // [4][hd]
  __shared__ float ms[4], ls[4];
  const int h = blockIdx.x, t = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int kvh = h / (Hq / Hkv);
  const int nkv = Hkv * hd;
  const int last = pos[t];
  const int* pt = page_table + (size_t)req[t] * max_pages;
  for (int i = threadIdx.x; i < hd; i += blockDim.x) qs[i] = to_f32(q[((size_t)t * Hq + h) * hd + i]);
  __syncthreads();
  float m = -INFINITY, l = 0.f, acc[MAXD];
#pragma unroll
  for (int i = 0; i < MAXD; ++i) acc[i] = 0.f;
  constexpr int VN = Vec16<KT>::N;
  for (int base = warp * 32; base <= last; base += 128) {
    const int p = base + lane;
    float s = -INFINITY;
    unsigned long long slot = 0;
    if (p <= last) {
      slot = (unsigned long long)pt[p / page_tokens] * page_tokens + (p % page_tokens);
      const KT* kr = kc + slot * nkv + (size_t)kvh * hd;
      float dot = 0.f;
      for (int d0 = 0; d0 < hd; d0 += VN) {
        float kv[VN];
        Vec16<KT>::load(kr + d0, kv);
#pragma unroll
        for (int j = 0; j < VN; ++j) dot = fmaf(qs[d0 + j], kv[j], dot);
      }
      s = dot * scale;
    }
    const float m_new = fmaxf(m, warp_max(s));
    const float pl = (p <= last) ? expf(s - m_new) : 0.f;
    const float corr = expf(m - m_new);  // exp(-inf) = 0 on the first chunk
    l = l * corr + warp_sum(pl);
#pragma unroll
    for (int i = 0; i < MAXD; ++i) acc[i] *= corr;
    m = m_new;
    const int cnt = min(32, last - base + 1);
    for (int j = 0; j < cnt; ++j) {
      const float pj = __shfl_sync(0xffffffffu, pl, j);
      const unsigned long long sj = __shfl_sync(0xffffffffu, slot, j);
      const KT* vr = vc + sj * nkv + (size_t)kvh * hd;
#pragma unroll
      for (int i = 0; i < MAXD; ++i) {
        const int d = lane + 32 * i;
        if (d < hd) acc[i] = fmaf(pj, to_f32(vr[d]), acc[i]);
      }
    }
  }
  if (lane == 0) { ms[warp] = m; ls[warp] = l; }
#pragma unroll
  for (int i = 0; i < MAXD; ++i) {
    const int d = lane + 32 * i;
    if (d < hd) accs[warp * hd + d] = acc[i];
  }
  __syncthreads();
  const float M = fmaxf(fmaxf(ms[0], ms[1]), fmaxf(ms[2], ms[3]));
  float L = 0.f;
#pragma unroll
  for (int w = 0; w < 4; ++w) L += ls[w] * expf(ms[w] - M);
  for (int d = threadIdx.x; d < hd; d += blockDim.x) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) v += accs[w * hd + d] * expf(ms[w] - M);
    o[((size_t)t * Hq + h) * hd + d] = from_f32<AT>(v / L);
  }
}

// Vocabulary-wide argmax of fp32 logits[T, V]: each block reduces a slice of one row to a
// packed (value, inverted index) key and merges it with a 64-bit atomic max.
__global__ void k_argmax(const float* __restrict__ logits, int V, int ld,
                         unsigned long long* __restrict__ keys) {
  __shared__ unsigned long long red[32];
  const int t = blockIdx.y;
  const int per = (V + gridDim.x - 1) / gridDim.x;
  const int lo = blockIdx.x * per, hi = min(V, lo + per);
  unsigned long long best = 0ull;
  for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) {
    const unsigned long long k = argmax_key(logits[(size_t)t * ld + i], (uint32_t)i);
    best = k > best ? k : best;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
    best = other > best ? other : best;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) red[warp] = best;
  __syncthreads();
  if (warp == 0) {
    best = (lane < (blockDim.x >> 5)) ? red[lane] : 0ull;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
      best = other > best ? other : best;
    }
    if (lane == 0 && best) atomicMax(keys + t, best);
  }
}

struct AcceptParams {
  int n_req;
  const int* val_req; const int* val_k; const int* val_off;
  const int* draft; int k_max;
  const unsigned long long* keys;
  int* target_tokens;  // [n_req, k_max+1]
  int* accept_len;     // [n_req]
  int commit;
  int* seq; int* n_seq; int max_seq_len;
};

// Stairs validation (paper Section 3.3, Fig. 5) on token ids: row 0 is ground truth; row r is
// kept while drafted token r-1 equals the main model's token for row r-1; accept_len is the
// number of kept rows after the first.  With commit, the kept drafts and the main model's
// token for the last kept row are appended to the request's sequence.
__global__ void k_accept(AcceptParams p) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= p.n_req) return;
  const int k = p.val_k[i], off = p.val_off[i], slot = p.val_req[i];
  int a = -1;
  for (int r = 0; r <= k; ++r) {
    const int tr = argmax_key_index(p.keys[off + r]);
    p.target_tokens[i * (p.k_max + 1) + r] = tr;
    if (a < 0 && r < k && p.draft[i * p.k_max + r] != tr) a = r;
  }
  if (a < 0) a = k;
  p.accept_len[i] = a;
  if (p.commit) {
    const int n = p.n_seq[slot];
    int* s = p.seq + (size_t)slot * p.max_seq_len;
    int w = n;
    for (int r = 0; r < a && w < p.max_seq_len; ++r) s[w++] = p.draft[i * p.k_max + r];
    if (w < p.max_seq_len) s[w++] = argmax_key_index(p.keys[off + a]);
    p.n_seq[slot] = w;
  }
}

// Assistant step epilogue: the argmax of one row becomes drafted token j.
__global__ void k_take_token(const unsigned long long* __restrict__ keys, int row, int* __restrict__ out, int j) {
  if (threadIdx.x == 0 && blockIdx.x == 0) out[j] = argmax_key_index(keys[row]);
}

}  // namespace stairs
