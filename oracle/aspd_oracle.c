/*
 * aspd_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 CPU statement of what ASPD's branch-isolated attention
 * step computes, written from the paper's equations.  It exists so that the
 * CUDA library can be checked against it.  Only the test-suite, the smoke
 * check and the benchmark's CPU-baseline leg may build, load or call it; the
 * product never does.  It shares no code, header, table or constant with the
 * CUDA path.
 *
 * Two forms of the same arithmetic:
 *
 *   dense      ("oracle-D")  Eq. 1-4 of the paper, literally, over a flat
 *              token list: positions from Eq. 4, visibility S from Eq. 3,
 *              mask from Eq. 2, masked softmax attention from Eq. 1.
 *   descriptor ("oracle-S")  the Hybrid Decoding Engine's statement of the
 *              same thing (Section 3.3): a parallel token attends the main
 *              branch (shared prefix) plus its own branch only, with
 *              sequentially increasing position IDs; after the segment the
 *              serial token attends the complete history and takes its actual
 *              index in the complete sequence as position.  This form works
 *              on a paged KV cache addressed through a page table.
 *
 * Readings of points the paper leaves open (each is also listed in the
 * design notes of the repository):
 *   - a token sees itself (Eq. 2 read as ordinary causal attention);
 *   - positions are 0-based (Eq. 4 is 1-based; RoPE scores depend only on
 *     differences of positions);
 *   - "delta i" of Eq. 4 is the index of the token inside its own branch;
 *   - stage_start is the number of tokens that precede the stage;
 *   - the positional encoding is RoPE with rotate-half pairing
 *     (x[i], x[i + d/2]) and inv_freq[i] = theta^(-2i/d);
 *   - query head h uses KV head floor(h / (Hq/Hkv));
 *   - masked keys get weight exactly 0 (additive -inf of Eq. 2).
 *
 * Pinning: every function here is pinned by CPU tests against closed forms,
 * library routines and a hand-derived worked example.  The paper prints no
 * attention output, mask or position table, so no pin is "a value the paper
 * prints"; parity against paper-printed values is unpinned for that reason
 * only.
 *
 * Everything is double precision.  Layouts are plain row-major:
 *   q      [n_tok][Hq ][d]
 *   k, v   [n_tok][Hkv][d]
 *   pools  [n_pages][Hkv][page_size][d]          (no swizzle, no packing)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_BAD (-1)

int aspd_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------ */
/* RoPE (reading: rotate-half pairing; theta is a parameter).                */
/* out may not alias x.                                                      */
/* ------------------------------------------------------------------------ */
void aspd_oracle_rope(const double* x, int d, double pos, double theta,
                      double* out) {
  int half = d / 2;
  for (int i = 0; i < half; ++i) {
    double inv_freq = pow(theta, -2.0 * (double)i / (double)d);
    double angle = pos * inv_freq;
    double c = cos(angle), s = sin(angle);
    out[i] = x[i] * c - x[i + half] * s;
    out[i + half] = x[i + half] * c + x[i] * s;
  }
}

/* ------------------------------------------------------------------------ */
/* Masked softmax attention of ONE query vector over a list of visible keys  */
/* (Eq. 1 with the -inf entries of Eq. 2 dropped: their weight is exactly 0).*/
/* Two passes: maximum, then exponentials and the weighted sum.              */
/* keys[j], vals[j] point at d doubles each.                                 */
/* ------------------------------------------------------------------------ */
static void attend_one(const double* qhat, int d, double sm_scale,
                       const double* const* keys, const double* const* vals,
                       long n_keys, double* logits, double* out) {
  double mx = -INFINITY;
  for (long j = 0; j < n_keys; ++j) {
    double s = 0.0;
    for (int e = 0; e < d; ++e) s += qhat[e] * keys[j][e];
    s *= sm_scale;
    logits[j] = s;
    if (s > mx) mx = s;
  }
  double denom = 0.0;
  for (int e = 0; e < d; ++e) out[e] = 0.0;
  for (long j = 0; j < n_keys; ++j) {
    double w = exp(logits[j] - mx);
    denom += w;
    for (int e = 0; e < d; ++e) out[e] += w * vals[j][e];
  }
  for (int e = 0; e < d; ++e) out[e] /= denom;
}

/* ======================================================================== */
/* oracle-D: dense, literal Eq. 1-4 over a flat token list                   */
/* ======================================================================== */

/*
 * Eq. 4.  Tokens are given in the flattened order of the sequence.
 *   branch[i] < 0  : token i is on the main branch (a serial stage)
 *   branch[i] >= 0 : token i belongs to that parallel branch of stage[i]
 * main token     : pos = number of tokens decoded before it = its flat index
 * parallel token : pos = stage_start + delta, stage_start = number of tokens
 *                  before the stage's first token, delta = index of the token
 *                  inside its own branch.
 */
int aspd_oracle_dense_positions(int L, const int* branch, const int* stage,
                                int* pos) {
  for (int i = 0; i < L; ++i) {
    if (branch[i] < 0) {
      pos[i] = i;
      continue;
    }
    int stage_start = -1;
    for (int j = 0; j < L; ++j)
      if (stage[j] == stage[i]) { stage_start = j; break; }
    int delta = 0;
    for (int j = 0; j < i; ++j)
      if (stage[j] == stage[i] && branch[j] == branch[i]) ++delta;
    pos[i] = stage_start + delta;
  }
  return ORACLE_OK;
}

/* Eq. 3: may query token i look at key token j at all? */
static int visibility_S(int i, int j, const int* branch, const int* stage) {
  if (branch[i] < 0) return 1;                                   /* main    */
  if (stage[i] == stage[j] && branch[i] == branch[j]) return 1;  /* same br */
  if (stage[i] != stage[j]) return 1;                            /* other stage */
  return 0;
}

/* Eq. 2 (with the self-visible reading): vis[i*L + j] = 1 iff M_ij = 0. */
int aspd_oracle_dense_visible(int L, const int* branch, const int* stage,
                              const int* pos, uint8_t* vis) {
  for (int i = 0; i < L; ++i)
    for (int j = 0; j < L; ++j) {
      int ok = visibility_S(i, j, branch, stage) && (pos[i] > pos[j] || i == j);
      vis[(size_t)i * L + j] = (uint8_t)(ok ? 1 : 0);
    }
  return ORACLE_OK;
}

/* The visible ("Shared") mask of the paper's attention-mask ablation: the visibility function is
 * 1 for every pair, so all that is left of Eq. 2 is the order of the position IDs -- token i
 * sees token j iff j's position precedes i's (and itself).  With the shared position IDs a
 * branch token at offset delta therefore sees the first delta tokens of EVERY branch of its stage:
 * exactly the tokens that exist when the branches decode in lockstep. */
int aspd_oracle_dense_visible_shared(int L, const int* pos, uint8_t* vis) {
  for (int i = 0; i < L; ++i)
    for (int j = 0; j < L; ++j)
      vis[(size_t)i * L + j] = (uint8_t)((pos[i] > pos[j] || i == j) ? 1 : 0);
  return ORACLE_OK;
}

/* Eq. 1 for every token of the flat list, every query head. */
static int dense_attn_impl(int L, int Hq, int Hkv, int d, double theta,
                           double sm_scale, const double* q, const double* k,
                           const double* v, const int* branch,
                           const int* stage, int shared_mask, double* out) {
  if (L <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv || d <= 0 || d % 2) return ORACLE_BAD;
  int G = Hq / Hkv;
  int* pos = (int*)malloc(sizeof(int) * L);
  uint8_t* vis = (uint8_t*)malloc((size_t)L * L);
  double* khat = (double*)malloc(sizeof(double) * (size_t)L * Hkv * d);
  aspd_oracle_dense_positions(L, branch, stage, pos);
  if (shared_mask) aspd_oracle_dense_visible_shared(L, pos, vis);
  else aspd_oracle_dense_visible(L, branch, stage, pos, vis);
  for (int j = 0; j < L; ++j)
    for (int h = 0; h < Hkv; ++h)
      aspd_oracle_rope(k + ((size_t)j * Hkv + h) * d, d, (double)pos[j], theta,
                       khat + ((size_t)j * Hkv + h) * d);
  const double** keys = (const double**)malloc(sizeof(double*) * L);
  const double** vals = (const double**)malloc(sizeof(double*) * L);
  double* logits = (double*)malloc(sizeof(double) * L);
  double* qhat = (double*)malloc(sizeof(double) * d);
  for (int i = 0; i < L; ++i)
    for (int hq = 0; hq < Hq; ++hq) {
      int h = hq / G;
      long n = 0;
      for (int j = 0; j < L; ++j)
        if (vis[(size_t)i * L + j]) {
          keys[n] = khat + ((size_t)j * Hkv + h) * d;
          vals[n] = v + ((size_t)j * Hkv + h) * d;
          ++n;
        }
      aspd_oracle_rope(q + ((size_t)i * Hq + hq) * d, d, (double)pos[i], theta, qhat);
      attend_one(qhat, d, sm_scale, keys, vals, n, logits,
                 out + ((size_t)i * Hq + hq) * d);
    }
  free(pos); free(vis); free(khat); free(keys); free(vals); free(logits); free(qhat);
  return ORACLE_OK;
}

int aspd_oracle_dense_attn(int L, int Hq, int Hkv, int d, double theta,
                           double sm_scale, const double* q, const double* k,
                           const double* v, const int* branch,
                           const int* stage, double* out) {
  return dense_attn_impl(L, Hq, Hkv, d, theta, sm_scale, q, k, v, branch, stage, 0, out);
}

/* Eq. 1 under the visible ("Shared") mask of the ablation. */
int aspd_oracle_dense_attn_shared(int L, int Hq, int Hkv, int d, double theta,
                                  double sm_scale, const double* q, const double* k,
                                  const double* v, const int* branch,
                                  const int* stage, double* out) {
  return dense_attn_impl(L, Hq, Hkv, d, theta, sm_scale, q, k, v, branch, stage, 1, out);
}

/* ======================================================================== */
/* oracle-S: descriptor form over a paged cache (Section 3.3)                */
/* ======================================================================== */
/*
 * A request r is described by plain integer arrays:
 *   prefix_len[r]    P: shared main-branch tokens at logical slots [0, P)
 *   n_branches[r]    N
 *   branch_begin[r]  first entry of the request in the br_* arrays
 *   page_begin[r]    first entry of the request in page_ids[]; logical slot s
 *                    of the request lives in physical page
 *                    page_ids[page_begin[r] + s / page_size], row s % page_size
 *   tail_off[r], tail_len[r]   main-branch tokens written after the segment
 *                    closed, at logical slots [tail_off, tail_off + tail_len)
 * and a branch b by
 *   br_kv_off[b]     first logical slot of the branch
 *   br_kv_len[b]     tokens of the branch in the cache AFTER this step's append
 *   br_q_len[b]      query tokens of the branch this step = its LAST q_len tokens;
 *                    0: a branch of the current stage that has finished (invisible to the others);
 *                    -1: a region of an EARLIER stage (a merged branch, or serial tokens written
 *                    between two parallel stages): Eq. 3's third case makes it visible to every
 *                    token of the current stage (the engine switches between serial and parallel
 *                    stages repeatedly, Section 3.3)
 *
 * mode 0 (parallel step): the new tokens are, request-major then branch-major,
 * the last q_len tokens of every branch.  mode 1 (serial step): one new token
 * per request, the last token of the tail.
 */
#define MODE_BRANCH 0
#define MODE_SERIAL 1
#define MASK_BRANCH_INVISIBLE 0   /* Eq. 2-3 */
#define MASK_SHARED 1             /* the ablation's visible mask */

/*
 * a1 + a2: position ID (Eq. 4) and logical slot of every new token.
 * Outputs have one entry per new token; returns their number, or -1.
 * req_out[t] = request of new token t.
 */
int aspd_oracle_new_tokens(int n_req, int mode, const int* prefix_len,
                           const int* n_branches, const int* branch_begin,
                           const int* tail_off, const int* tail_len,
                           const int* br_kv_off, const int* br_kv_len,
                           const int* br_q_len, int* pos_out, int* slot_out,
                           int* req_out) {
  int n = 0;
  for (int r = 0; r < n_req; ++r) {
    int P = prefix_len[r];
    if (mode == MODE_BRANCH) {
      int stage_start = P;                        /* tokens before the stage: prefix + earlier stages */
      for (int b = 0; b < n_branches[r]; ++b)
        if (br_q_len[branch_begin[r] + b] == -1) stage_start += br_kv_len[branch_begin[r] + b];
      for (int b = 0; b < n_branches[r]; ++b) {
        int B = branch_begin[r] + b;
        for (int i = 0; i < br_q_len[B]; ++i) {
          int k = br_kv_len[B] - br_q_len[B] + i; /* index inside the branch */
          if (k < 0) return ORACLE_BAD;
          pos_out[n] = stage_start + k;           /* stage_start + delta     */
          slot_out[n] = br_kv_off[B] + k;
          req_out[n] = r;
          ++n;
        }
      }
    } else {
      /* actual index in the complete sequence: every token that is already
         in the cache counts, whichever branch holds it */
      int total = P;
      for (int b = 0; b < n_branches[r]; ++b) total += br_kv_len[branch_begin[r] + b];
      if (tail_len[r] < 1) return ORACLE_BAD;
      pos_out[n] = total + tail_len[r] - 1;
      slot_out[n] = tail_off[r] + tail_len[r] - 1;
      req_out[n] = r;
      ++n;
    }
  }
  return n;
}

/*
 * a3: K' = RoPE(K, pos), V' = V, scattered into the paged pools.
 * k_new, v_new [n_new][Hkv][d]; pools [n_pool_pages][Hkv][page_size][d].
 */
int aspd_oracle_kv_append(int n_new, int Hkv, int d, int page_size,
                          double theta, const double* k_new,
                          const double* v_new, const int* pos, const int* req,
                          const int* slot, const int* page_begin,
                          const int* page_ids, double* k_pool, double* v_pool) {
  for (int t = 0; t < n_new; ++t) {
    int page = page_ids[page_begin[req[t]] + slot[t] / page_size];
    int row = slot[t] % page_size;
    for (int h = 0; h < Hkv; ++h) {
      size_t dst = (((size_t)page * Hkv + h) * page_size + row) * d;
      aspd_oracle_rope(k_new + ((size_t)t * Hkv + h) * d, d, (double)pos[t], theta,
                       k_pool + dst);
      memcpy(v_pool + dst, v_new + ((size_t)t * Hkv + h) * d, sizeof(double) * d);
    }
  }
  return ORACLE_OK;
}

/* Read one cached token back (logical slot -> page table -> row). */
static const double* cached(const double* pool, const int* page_ids, int pbeg,
                            int slot, int h, int Hkv, int page_size, int d) {
  int page = page_ids[pbeg + slot / page_size];
  int row = slot % page_size;
  return pool + (((size_t)page * Hkv + h) * page_size + row) * d;
}

/*
 * a4-a7 (mode 0) and a9 (mode 1): attention of every new token.
 * q [n_new][Hq][d] raw (un-rotated); the query is rotated here at the same
 * position as the token's own key.  out [n_new][Hq][d].
 *
 * Visible set of a parallel token (branch B, i-th of its q_len queries):
 *   the prefix [0, P)  and  tokens 0 .. kv_len - q_len + i of branch B.
 * Visible set of the serial token: prefix, every token of every branch, and
 * the tail up to and including itself.
 */
static int attn_impl(int n_req, int mode, int Hq, int Hkv, int d,
                     int page_size, double theta, double sm_scale,
                     const int* prefix_len, const int* n_branches,
                     const int* branch_begin, const int* page_begin,
                     const int* tail_off, const int* tail_len,
                     const int* br_kv_off, const int* br_kv_len,
                     const int* br_q_len, const int* page_ids, const double* q,
                     const int* q_pos_given, int mask_mode,
                     const double* k_pool, const double* v_pool, double* out) {
  if (Hq % Hkv || d % 2) return ORACLE_BAD;
  int G = Hq / Hkv;
  /* enumerate the new tokens: (request, branch or -1, index in branch) */
  int cap = 0;
  for (int r = 0; r < n_req; ++r) {
    if (mode == MODE_SERIAL) cap += 1;
    else for (int b = 0; b < n_branches[r]; ++b) cap += br_q_len[branch_begin[r] + b] > 0 ? br_q_len[branch_begin[r] + b] : 0;
  }
  int* t_req = (int*)malloc(sizeof(int) * (cap + 1));
  int* t_br = (int*)malloc(sizeof(int) * (cap + 1));
  int* t_k = (int*)malloc(sizeof(int) * (cap + 1));
  int* t_pos0 = (int*)malloc(sizeof(int) * (cap + 1));   /* stage_start of the token's stage */
  int n = 0;
  long max_keys = 0;
  for (int r = 0; r < n_req; ++r) {
    long total = prefix_len[r];
    for (int b = 0; b < n_branches[r]; ++b) total += br_kv_len[branch_begin[r] + b];
    total += tail_len ? tail_len[r] : 0;
    if (total > max_keys) max_keys = total;
    if (mode == MODE_SERIAL) {
      t_req[n] = r; t_br[n] = -1; t_k[n] = 0; t_pos0[n] = 0; ++n;
    } else {
      for (int b = 0; b < n_branches[r]; ++b) {
        int B = branch_begin[r] + b;
        for (int i = 0; i < br_q_len[B]; ++i) {
          int stage_start = prefix_len[r];        /* tokens before the stage: prefix + earlier stages */
          for (int c = 0; c < n_branches[r]; ++c)
            if (br_q_len[branch_begin[r] + c] == -1) stage_start += br_kv_len[branch_begin[r] + c];
          t_req[n] = r; t_br[n] = B; t_k[n] = br_kv_len[B] - br_q_len[B] + i; t_pos0[n] = stage_start; ++n;
        }
      }
    }
  }
  int fail = 0;
#pragma omp parallel
  {
    const double** keys = (const double**)malloc(sizeof(double*) * (max_keys + 1));
    const double** vals = (const double**)malloc(sizeof(double*) * (max_keys + 1));
    double* logits = (double*)malloc(sizeof(double) * (max_keys + 1));
    double* qhat = (double*)malloc(sizeof(double) * d);
#pragma omp for collapse(2) schedule(dynamic, 1)
    for (int t = 0; t < n; ++t)
      for (int hq = 0; hq < Hq; ++hq) {
        int r = t_req[t], h = hq / G, P = prefix_len[r], pb = page_begin[r];
        long m = 0;
        int qpos;
        for (int s = 0; s < P; ++s) {
          keys[m] = cached(k_pool, page_ids, pb, s, h, Hkv, page_size, d);
          vals[m] = cached(v_pool, page_ids, pb, s, h, Hkv, page_size, d);
          ++m;
        }
        if (mode == MODE_BRANCH) {
          int B = t_br[t];
          for (int b = 0; b < n_branches[r]; ++b) {        /* regions of earlier stages */
            int S = branch_begin[r] + b;
            if (br_q_len[S] != -1) continue;
            for (int j = 0; j < br_kv_len[S]; ++j) {
              int s = br_kv_off[S] + j;
              keys[m] = cached(k_pool, page_ids, pb, s, h, Hkv, page_size, d);
              vals[m] = cached(v_pool, page_ids, pb, s, h, Hkv, page_size, d);
              ++m;
            }
          }
          for (int j = 0; j <= t_k[t]; ++j) {
            int s = br_kv_off[B] + j;
            keys[m] = cached(k_pool, page_ids, pb, s, h, Hkv, page_size, d);
            vals[m] = cached(v_pool, page_ids, pb, s, h, Hkv, page_size, d);
            ++m;
          }
          if (mask_mode == MASK_SHARED) {                  /* the other branches of the stage, at smaller offsets */
            for (int b = 0; b < n_branches[r]; ++b) {
              int C = branch_begin[r] + b;
              if (C == B || br_q_len[C] == -1) continue;
              for (int j = 0; j < br_kv_len[C] && j < t_k[t]; ++j) {
                int s = br_kv_off[C] + j;
                keys[m] = cached(k_pool, page_ids, pb, s, h, Hkv, page_size, d);
                vals[m] = cached(v_pool, page_ids, pb, s, h, Hkv, page_size, d);
                ++m;
              }
            }
          }
          qpos = t_pos0[t] + t_k[t];
        } else {
          int total = P;
          for (int b = 0; b < n_branches[r]; ++b) {
            int B = branch_begin[r] + b;
            total += br_kv_len[B];
            for (int j = 0; j < br_kv_len[B]; ++j) {
              int s = br_kv_off[B] + j;
              keys[m] = cached(k_pool, page_ids, pb, s, h, Hkv, page_size, d);
              vals[m] = cached(v_pool, page_ids, pb, s, h, Hkv, page_size, d);
              ++m;
            }
          }
          if (tail_len[r] < 1) { fail = 1; continue; }
          for (int j = 0; j < tail_len[r]; ++j) {
            int s = tail_off[r] + j;
            keys[m] = cached(k_pool, page_ids, pb, s, h, Hkv, page_size, d);
            vals[m] = cached(v_pool, page_ids, pb, s, h, Hkv, page_size, d);
            ++m;
          }
          qpos = total + tail_len[r] - 1;
        }
        if (q_pos_given) qpos = q_pos_given[t];   /* a position-ID variant: the caller's rule, not Eq. 4 */
        aspd_oracle_rope(q + ((size_t)t * Hq + hq) * d, d, (double)qpos, theta, qhat);
        attend_one(qhat, d, sm_scale, keys, vals, m, logits,
                   out + ((size_t)t * Hq + hq) * d);
      }
    free(keys); free(vals); free(logits); free(qhat);
  }
  free(t_req); free(t_br); free(t_k); free(t_pos0);
  return fail ? ORACLE_BAD : ORACLE_OK;
}

int aspd_oracle_attn(int n_req, int mode, int Hq, int Hkv, int d,
                     int page_size, double theta, double sm_scale,
                     const int* prefix_len, const int* n_branches,
                     const int* branch_begin, const int* page_begin,
                     const int* tail_off, const int* tail_len,
                     const int* br_kv_off, const int* br_kv_len,
                     const int* br_q_len, const int* page_ids, const double* q,
                     const double* k_pool, const double* v_pool, double* out) {
  return attn_impl(n_req, mode, Hq, Hkv, d, page_size, theta, sm_scale, prefix_len, n_branches, branch_begin,
                   page_begin, tail_off, tail_len, br_kv_off, br_kv_len, br_q_len, page_ids, q, 0, MASK_BRANCH_INVISIBLE, k_pool, v_pool, out);
}

/*
 * The same attention with the query positions given by the caller instead of Eq. 4: the
 * position-ID variants of the paper's ablation (pre-allocated fixed-length intervals per branch;
 * "Same-Max": the serial token resumes at the largest branch position).  Masking is unchanged;
 * the keys carry whatever positions they were appended with.
 */
int aspd_oracle_attn_at(int n_req, int mode, int Hq, int Hkv, int d,
                        int page_size, double theta, double sm_scale,
                        const int* prefix_len, const int* n_branches,
                        const int* branch_begin, const int* page_begin,
                        const int* tail_off, const int* tail_len,
                        const int* br_kv_off, const int* br_kv_len,
                        const int* br_q_len, const int* page_ids, const double* q,
                        const int* q_pos,
                        const double* k_pool, const double* v_pool, double* out) {
  if (!q_pos) return ORACLE_BAD;
  return attn_impl(n_req, mode, Hq, Hkv, d, page_size, theta, sm_scale, prefix_len, n_branches, branch_begin,
                   page_begin, tail_off, tail_len, br_kv_off, br_kv_len, br_q_len, page_ids, q, q_pos, MASK_BRANCH_INVISIBLE, k_pool, v_pool, out);
}

/* The same with the mask of the attention-mask ablation chosen by mask_mode (q_pos may be null). */
int aspd_oracle_attn_masked(int n_req, int mode, int Hq, int Hkv, int d,
                            int page_size, double theta, double sm_scale,
                            const int* prefix_len, const int* n_branches,
                            const int* branch_begin, const int* page_begin,
                            const int* tail_off, const int* tail_len,
                            const int* br_kv_off, const int* br_kv_len,
                            const int* br_q_len, const int* page_ids, const double* q,
                            const int* q_pos, int mask_mode,
                            const double* k_pool, const double* v_pool, double* out) {
  if (mask_mode != MASK_BRANCH_INVISIBLE && mask_mode != MASK_SHARED) return ORACLE_BAD;
  return attn_impl(n_req, mode, Hq, Hkv, d, page_size, theta, sm_scale, prefix_len, n_branches, branch_begin,
                   page_begin, tail_off, tail_len, br_kv_off, br_kv_len, br_q_len, page_ids, q, q_pos, mask_mode, k_pool, v_pool, out);
}

/*
 * The set of logical slots a new token may look at, as the descriptor form
 * defines it (integers only; used to compare mask membership bit for bit).
 * vis_out [n_new][n_slots] (0/1); n_slots = slots per request row given.
 */
static int visible_slots_impl(int n_req, int mode, int n_slots,
                              const int* prefix_len, const int* n_branches,
                              const int* branch_begin, const int* tail_off,
                              const int* tail_len, const int* br_kv_off,
                              const int* br_kv_len, const int* br_q_len,
                              int mask_mode, uint8_t* vis_out) {
  int n = 0;
  for (int r = 0; r < n_req; ++r) {
    int P = prefix_len[r];
    if (mode == MODE_BRANCH) {
      for (int b = 0; b < n_branches[r]; ++b) {
        int B = branch_begin[r] + b;
        for (int i = 0; i < br_q_len[B]; ++i) {
          uint8_t* row = vis_out + (size_t)n * n_slots;
          memset(row, 0, n_slots);
          for (int s = 0; s < P; ++s) row[s] = 1;
          for (int c = 0; c < n_branches[r]; ++c) {
            int S = branch_begin[r] + c;
            if (br_q_len[S] == -1) for (int j = 0; j < br_kv_len[S]; ++j) row[br_kv_off[S] + j] = 1;
          }
          for (int j = 0; j <= br_kv_len[B] - br_q_len[B] + i; ++j) row[br_kv_off[B] + j] = 1;
          if (mask_mode == MASK_SHARED)                     /* other branches of the stage: offsets below the token's own */
            for (int c = 0; c < n_branches[r]; ++c) {
              int C = branch_begin[r] + c;
              if (C == B || br_q_len[C] == -1) continue;
              for (int j = 0; j < br_kv_len[C] && j < br_kv_len[B] - br_q_len[B] + i; ++j) row[br_kv_off[C] + j] = 1;
            }
          ++n;
        }
      }
    } else {
      uint8_t* row = vis_out + (size_t)n * n_slots;
      memset(row, 0, n_slots);
      for (int s = 0; s < P; ++s) row[s] = 1;
      for (int b = 0; b < n_branches[r]; ++b) {
        int B = branch_begin[r] + b;
        for (int j = 0; j < br_kv_len[B]; ++j) row[br_kv_off[B] + j] = 1;
      }
      for (int j = 0; j < tail_len[r]; ++j) row[tail_off[r] + j] = 1;
      ++n;
    }
  }
  return n;
}

int aspd_oracle_visible_slots(int n_req, int mode, int n_slots,
                              const int* prefix_len, const int* n_branches,
                              const int* branch_begin, const int* tail_off,
                              const int* tail_len, const int* br_kv_off,
                              const int* br_kv_len, const int* br_q_len,
                              uint8_t* vis_out) {
  return visible_slots_impl(n_req, mode, n_slots, prefix_len, n_branches, branch_begin, tail_off, tail_len, br_kv_off,
                            br_kv_len, br_q_len, MASK_BRANCH_INVISIBLE, vis_out);
}

int aspd_oracle_visible_slots_masked(int n_req, int mode, int n_slots,
                                     const int* prefix_len, const int* n_branches,
                                     const int* branch_begin, const int* tail_off,
                                     const int* tail_len, const int* br_kv_off,
                                     const int* br_kv_len, const int* br_q_len,
                                     int mask_mode, uint8_t* vis_out) {
  if (mask_mode != MASK_BRANCH_INVISIBLE && mask_mode != MASK_SHARED) return ORACLE_BAD;
  return visible_slots_impl(n_req, mode, n_slots, prefix_len, n_branches, branch_begin, tail_off, tail_len, br_kv_off,
                            br_kv_len, br_q_len, mask_mode, vis_out);
}
