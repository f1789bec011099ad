/*
 * CPU oracle for the blockwise verification step of trajectory-level
 * speculative decoding for diffusion language models.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow,
 * fp64 restatement of what the verification step computes, written from the
 * paper's definitions.  It shares no code with the CUDA library; only tests,
 * the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Inputs that the GPU receives as bf16 or fp32 arrive here as fp32 arrays
 * (both widen to fp32 exactly); all arithmetic below is in double.
 *
 * Parts, and the passage each follows:
 *   oracle_dense_mask        Section 3.3, the two visibility rules + "bidirectional"
 *   oracle_masked_attention  Section 3.3 / App. A: softmax attention under that mask
 *   oracle_confidence_topk   Eq. 2 (confidence) and the top-k candidates of Section 3.2
 *   oracle_decode_rule       Alg. 1 Phase 1 (H = {conf > tau}) with the top-1
 *                            fallback of Eqs. 6-7
 *   oracle_accept            Section 3.3 "Verification procedure" (greedy / longest path;
 *                            exact, top-1, top-k-membership and probability tests)
 *   oracle_draft_token_prob  probability of a drafted token under its parent (Eq. 2's softmax)
 *   oracle_build_draft_tree  Alg. 1 Phase 2 (the step before the path; built after it)
 *
 * Pins (tests/test_oracle_*.py): textbook attention for one branch, plain
 * bidirectional attention for an all-visible mask, per-row brute force,
 * closed forms, hand-worked acceptance trees, and the exactness theorem
 * (Theorem 1) on a toy model.  The paper prints no numeric value for this
 * path, so parity against printed values is unpinned; parity is against the
 * definitions and invariants listed above.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------
 * Section 3.3.  Keys are laid out as [cached prefix+suffix tokens | draft rows
 * of branch 0 | draft rows of branch 1 | ...].  Query row i belongs to branch
 * b = i / R.  Rule 1: every row of a draft block sees all cached tokens
 * (those below cache_lens[s] when a sequence holds fewer than Nc).  Rule 2:
 * it sees no row of another draft block.  "Bidirectional" inside the block:
 * it sees every row of its own block, itself included.  A caller-supplied
 * bitset vis[s][b] (bit j = branch b may read branch j) generalises rule 2;
 * the own-branch bit is always taken as set.
 * ---------------------------------------------------------------------- */
void oracle_dense_mask(int S, int B, int R, int Nc, const uint64_t* vis,
                       const int32_t* cache_lens, uint8_t* mask) {
  const int N = B * R;
  const int W = (B + 63) / 64;
  const int64_t L = (int64_t)Nc + N;
  for (int s = 0; s < S; ++s) {
    const int clen = cache_lens ? cache_lens[s] : Nc;
    for (int i = 0; i < N; ++i) {
      uint8_t* row = mask + ((int64_t)s * N + i) * L;
      const int b = i / R;
      for (int j = 0; j < Nc; ++j) row[j] = (uint8_t)(j < clen);
      for (int j = 0; j < N; ++j) {
        const int bj = j / R;
        int visible = (bj == b);
        if (vis && !visible) {
          const uint64_t w = vis[((int64_t)s * B + b) * W + bj / 64];
          visible = (int)((w >> (bj % 64)) & 1u);
        }
        row[Nc + j] = (uint8_t)visible;
      }
    }
  }
}

/* ------------------------------------------------------------------------
 * Masked softmax attention, one (sequence, head, draft row) at a time.
 *   a_j  = sm_scale * <q_i, k_j>        for visible j
 *   O_i  = sum_j exp(a_j - max a) v_j / sum_j exp(a_j - max a)
 *   lse  = max a + log sum_j exp(a_j - max a)
 * Grouped-query heads: query head h reads kv head h / (Hq / Hkv).
 * Layouts (contiguous): q,out [S,N,Hq,d]; kc,vc [S,Nc,Hkv,d]; kd,vd [S,N,Hkv,d];
 * mask [S,N,Nc+N]; lse [S,Hq,N] (nullable).
 * ---------------------------------------------------------------------- */
void oracle_masked_attention(int S, int N, int Nc, int Hq, int Hkv, int d,
                             const float* q, const float* kc, const float* vc,
                             const float* kd, const float* vd,
                             const uint8_t* mask, double sm_scale, double* out,
                             double* lse) {
  const int64_t L = (int64_t)Nc + N;
  const int group = Hq / Hkv;
  const int64_t total = (int64_t)S * Hq * N;
#pragma omp parallel
  {
    double* a = (double*)malloc(sizeof(double) * (size_t)L);
    double* acc = (double*)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 8)
    for (int64_t t = 0; t < total; ++t) {
      const int i = (int)(t % N);
      const int h = (int)((t / N) % Hq);
      const int s = (int)(t / ((int64_t)N * Hq));
      const int g = h / group;
      const uint8_t* mrow = mask + ((int64_t)s * N + i) * L;
      const float* qi = q + (((int64_t)s * N + i) * Hq + h) * d;
      double amax = -INFINITY;
      for (int64_t j = 0; j < L; ++j) {
        if (!mrow[j]) continue;
        const float* kj = (j < Nc)
                              ? kc + (((int64_t)s * Nc + j) * Hkv + g) * d
                              : kd + (((int64_t)s * N + (j - Nc)) * Hkv + g) * d;
        double dot = 0.0;
        for (int c = 0; c < d; ++c) dot += (double)qi[c] * (double)kj[c];
        a[j] = sm_scale * dot;
        if (a[j] > amax) amax = a[j];
      }
      double z = 0.0;
      for (int c = 0; c < d; ++c) acc[c] = 0.0;
      for (int64_t j = 0; j < L; ++j) {
        if (!mrow[j]) continue;
        const float* vj = (j < Nc)
                              ? vc + (((int64_t)s * Nc + j) * Hkv + g) * d
                              : vd + (((int64_t)s * N + (j - Nc)) * Hkv + g) * d;
        const double p = exp(a[j] - amax);
        z += p;
        for (int c = 0; c < d; ++c) acc[c] += p * (double)vj[c];
      }
      double* oi = out + (((int64_t)s * N + i) * Hq + h) * d;
      for (int c = 0; c < d; ++c) oi[c] = acc[c] / z;
      if (lse) lse[((int64_t)s * Hq + h) * N + i] = amax + log(z);
    }
    free(a);
    free(acc);
  }
}

/* ------------------------------------------------------------------------
 * Eq. 2 and the candidate pool of Section 3.2.  Per row of logits l[0..V):
 *   m = max l,  Z = sum exp(l - m),  p_v = exp(l_v - m) / Z,
 *   conf = max_v p_v = p of the first candidate,
 *   candidates = the first k vocabulary entries in the order
 *                (logit descending, index ascending),
 *   lse = m + log Z.
 * The order is decided on the raw input values, so the indices are unique.
 * Selection is k plain scans: scan t picks the best entry that comes
 * strictly after the previous pick in that order.
 * ---------------------------------------------------------------------- */
static int comes_before(float va, int ia, float vb, int ib) {
  /* 1 if (va, ia) precedes (vb, ib): larger logit first, then lower index */
  if (va > vb) return 1;
  if (va < vb) return 0;
  return ia < ib;
}

void oracle_confidence_topk(const float* logits, int64_t n_rows, int V,
                            int64_t row_stride, int k, double* conf,
                            int32_t* topk_idx, double* topk_prob, double* lse) {
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t r = 0; r < n_rows; ++r) {
    const float* l = logits + r * row_stride;
    double m = -INFINITY;
    for (int v = 0; v < V; ++v)
      if ((double)l[v] > m) m = (double)l[v];
    double z = 0.0;
    for (int v = 0; v < V; ++v) z += exp((double)l[v] - m);
    int have_prev = 0, prev_i = -1;
    float prev_v = 0.0f;
    for (int t = 0; t < k; ++t) {
      int best = -1;
      for (int v = 0; v < V; ++v) {
        if (have_prev && !comes_before(prev_v, prev_i, l[v], v)) continue;
        if (best < 0 || comes_before(l[v], v, l[best], best)) best = v;
      }
      topk_idx[r * k + t] = best;
      topk_prob[r * k + t] = exp((double)l[best] - m) / z;
      have_prev = 1;
      prev_v = l[best];
      prev_i = best;
    }
    conf[r] = topk_prob[r * k]; /* Eq. 2: the probability of the first candidate */
    if (lse) lse[r] = m + log(z);
  }
}

/* ------------------------------------------------------------------------
 * Decode rule U(p) for one node (block state of R rows): what threshold
 * ("sequential confidence") decoding would unmask next, given the node's
 * per-row confidence and top-1 token.
 *   M = rows still holding mask_id
 *   H = {r in M : conf[r] > tau}                      (Alg. 1, Phase 1: strict >)
 *   U = {(r, top1[r]) : r in H}                       if H is not empty
 *   U = {(r*, top1[r*])}, r* = argmax_{r in M} conf   otherwise (Eqs. 6-7;
 *                                                      lowest row on ties)
 *   U = {}                                            if M is empty
 * conf is the fp32 value the interface carries.  flag[r] = 1 for rows in U.
 * Returns |U|.
 * ---------------------------------------------------------------------- */
int oracle_decode_rule(int R, const int32_t* state, int32_t mask_id,
                       const float* conf, const int32_t* top1, float tau,
                       uint8_t* flag, int32_t* tok) {
  int n_high = 0, n_masked = 0, best = -1;
  for (int r = 0; r < R; ++r) {
    flag[r] = 0;
    tok[r] = -1;
  }
  for (int r = 0; r < R; ++r) {
    if (state[r] != mask_id) continue;
    ++n_masked;
    if (best < 0 || conf[r] > conf[best]) best = r;
    if (conf[r] > tau) {
      flag[r] = 1;
      tok[r] = top1[r];
      ++n_high;
    }
  }
  if (n_high > 0) return n_high;
  if (n_masked == 0) return 0;
  flag[best] = 1;
  tok[best] = top1[best];
  return 1;
}

/* ------------------------------------------------------------------------
 * Acceptance (Section 3.3, "Verification procedure").
 * Tree: parent[s][b] (parent[0] = -1, parent[b] < b), node 0 = root.
 * Edge parent->c carries the delta D(c) = rows the parent had masked and c
 * has filled, with c's tokens.  c is malformed if it alters a row the parent
 * had already filled or re-masks one; a malformed or empty delta is invalid.
 *   rule 0 (EXACT): D(c) == U(parent) as sets of (row, token)
 *   rule 1 (TOP1) : every (r, t) in D(c) has t == top1[parent][r]
 *   rule 2 (TOPK) : every (r, t) in D(c) has t among the parent's topk_m most
 *                   probable tokens at r (the top-k-membership alternative)
 *   rule 3 (PROB) : every (r, t) in D(c) has draft_prob[c][r] > tau, where
 *                   draft_prob[c][r] is the probability the parent's
 *                   distribution at r gives to t (the probability-above-tau
 *                   alternative; strict, as in Alg. 1)
 * Rules 1-3 admit trajectory drift (Section 4, last paragraph); only rule 0
 * is the test of Theorem 1.  top1 holds, per (node, row), the candidate
 * tokens in descending probability, top1_stride apart; entry 0 is the arg-max.
 * An edge whose parent index lies outside [0, c) is not an edge of the tree:
 * it is invalid and c counts as a depth-1 node with no valid prefix.
 * prefix_len[b] = number of leading valid edges on the path root -> b.
 * search 0 (GREEDY): from the root, move to the lowest-index valid child
 *                    until there is none.
 * search 1 (LONGEST): the deepest node whose whole path is valid, lowest
 *                    index among equals.
 * Outputs per sequence: accepted node, its depth, tokens it holds beyond the
 * root, and U(accepted node) for the caller's next root.
 * ---------------------------------------------------------------------- */
void oracle_accept(int S, int B, int R, const int32_t* parent,
                   const int32_t* state, int32_t mask_id, const float* conf,
                   const int32_t* top1, int64_t top1_stride, int topk_m,
                   const float* draft_prob, float tau,
                   int rule, int search, uint8_t* edge_valid,
                   int32_t* prefix_len, int32_t* accepted_node,
                   int32_t* accepted_len, int32_t* n_new_tokens,
                   uint8_t* unmask_flag, int32_t* unmask_tok) {
  uint8_t* uflag = (uint8_t*)malloc((size_t)R);
  int32_t* utok = (int32_t*)malloc(sizeof(int32_t) * (size_t)R);
  int32_t* t1 = (int32_t*)malloc(sizeof(int32_t) * (size_t)R);
  int32_t* depth = (int32_t*)malloc(sizeof(int32_t) * (size_t)B);
  for (int s = 0; s < S; ++s) {
    const int32_t* par = parent + (int64_t)s * B;
    uint8_t* ev = edge_valid + (int64_t)s * B;
    int32_t* pl = prefix_len + (int64_t)s * B;
    ev[0] = 1;
    pl[0] = 0;
    depth[0] = 0;
    for (int c = 1; c < B; ++c) {
      const int p = par[c];
      if (p < 0 || p >= c) {
        ev[c] = 0;
        depth[c] = 1;
        pl[c] = 0;
        continue;
      }
      const int32_t* sp = state + ((int64_t)s * B + p) * R;
      const int32_t* sc = state + ((int64_t)s * B + c) * R;
      const float* cp = conf + ((int64_t)s * B + p) * R;
      for (int r = 0; r < R; ++r)
        t1[r] = top1[(((int64_t)s * B + p) * R + r) * top1_stride];
      oracle_decode_rule(R, sp, mask_id, cp, t1, tau, uflag, utok);
      int n_delta = 0, malformed = 0, ok = 1;
      for (int r = 0; r < R; ++r) {
        const int p_masked = (sp[r] == mask_id);
        const int c_masked = (sc[r] == mask_id);
        if (!p_masked) {
          if (sc[r] != sp[r]) malformed = 1;
          continue;
        }
        if (c_masked) {
          if (rule == 0 && uflag[r]) ok = 0; /* U has a row the delta lacks */
          continue;
        }
        ++n_delta;
        if (rule == 0) {
          if (!uflag[r] || utok[r] != sc[r]) ok = 0;
        } else if (rule == 1) {
          if (t1[r] != sc[r]) ok = 0;
        } else if (rule == 2) {
          const int32_t* cand = top1 + (((int64_t)s * B + p) * R + r) * top1_stride;
          int found = 0;
          for (int j = 0; j < topk_m; ++j) found |= (cand[j] == sc[r]);
          if (!found) ok = 0;
        } else {
          if (!(draft_prob[((int64_t)s * B + c) * R + r] > tau)) ok = 0;
        }
      }
      ev[c] = (uint8_t)(ok && !malformed && n_delta > 0);
      depth[c] = depth[p] + 1;
      pl[c] = (pl[p] == depth[p] && ev[c]) ? depth[c] : pl[p];
    }
    int acc = 0;
    if (search == 0) {
      for (;;) {
        int next = -1;
        for (int c = 1; c < B; ++c)
          if (par[c] == acc && ev[c]) {
            next = c;
            break;
          }
        if (next < 0) break;
        acc = next;
      }
    } else {
      for (int b = 1; b < B; ++b)
        if (pl[b] == depth[b] && depth[b] > depth[acc]) acc = b;
    }
    accepted_node[s] = acc;
    accepted_len[s] = depth[acc];
    const int32_t* s0 = state + ((int64_t)s * B) * R;
    const int32_t* sa = state + ((int64_t)s * B + acc) * R;
    int f0 = 0, fa = 0;
    for (int r = 0; r < R; ++r) {
      f0 += (s0[r] != mask_id);
      fa += (sa[r] != mask_id);
    }
    n_new_tokens[s] = fa - f0;
    for (int r = 0; r < R; ++r)
      t1[r] = top1[(((int64_t)s * B + acc) * R + r) * top1_stride];
    oracle_decode_rule(R, sa, mask_id, conf + ((int64_t)s * B + acc) * R, t1,
                       tau, unmask_flag + (int64_t)s * R,
                       unmask_tok + (int64_t)s * R);
  }
  free(uflag);
  free(utok);
  free(t1);
  free(depth);
}

/* ------------------------------------------------------------------------
 * Probability of every drafted token under its parent's distribution
 * (the quantity the probability-above-tau reading of Section 3.3 tests): for child c,
 * row r in D(c) with token t,
 *   out[c][r] = exp(z_t - max z) / sum_v exp(z_v - max z),  z = logits[parent(c)][r]
 * (Eq. 2's softmax).  Rows outside D(c), the root, nodes with a parent index
 * outside [0, c) and tokens outside [0, V) get 0.
 * logits [S,B,R,V] fp32, out [S,B,R] fp64.
 * ---------------------------------------------------------------------- */
void oracle_draft_token_prob(int S, int B, int R, int V, const float* logits,
                             const int32_t* parent, const int32_t* state,
                             int32_t mask_id, double* out) {
  for (int s = 0; s < S; ++s)
    for (int c = 0; c < B; ++c) {
      const int p = parent[(int64_t)s * B + c];
      for (int r = 0; r < R; ++r) {
        double* o = out + ((int64_t)s * B + c) * R + r;
        *o = 0.0;
        if (c == 0 || p < 0 || p >= c) continue;
        const int32_t tp = state[((int64_t)s * B + p) * R + r];
        const int32_t tc = state[((int64_t)s * B + c) * R + r];
        if (tp != mask_id || tc == mask_id || tc < 0 || tc >= V) continue;
        const float* z = logits + (((int64_t)s * B + p) * R + r) * (int64_t)V;
        double zmax = -INFINITY, sum = 0.0;
        for (int v = 0; v < V; ++v)
          if ((double)z[v] > zmax) zmax = (double)z[v];
        for (int v = 0; v < V; ++v) sum += exp((double)z[v] - zmax);
        *o = exp((double)z[tc] - zmax) / sum;
      }
    }
}

/* ------------------------------------------------------------------------
 * Alg. 1, Phase 2 (speculative expansion) for one sequence.  The root block
 * state is given (Phase 1, filling the rows above tau, is what the caller
 * does with the previous step's unmask set); the candidate pool of Section 3.2
 * is the top-k (token, probability) of every row that is still masked in the
 * root, taken from the scores of the previous verification pass.
 *
 * The paper names but does not define GenerateTopK, GenerateTop1 and
 * PruneByConfidence; the reading implemented here:
 *   level 1  (GenerateTopK): the k best pool entries (row, j) by probability
 *            (ties: lower row, then lower rank j), one child per entry =
 *            root + that one (row, token);
 *   level >1 (GenerateTop1): every frontier node gets one child = the node +
 *            the best pool entry whose row is still masked in that node;
 *   PruneByConfidence: keep the W children of a level whose added entry has
 *            the largest probability (ties: earlier in generation order), in
 *            that order; they become the next frontier;
 *   the tree holds at most max_nodes nodes (the "n child blocks" of the
 *   WxDy(n) naming, plus the root): a level is cut where the budget ends.
 * Nodes are numbered level by level in pruned order, so siblings are listed in
 * descending draft confidence.  Unused node slots are copies of the root with
 * parent 0 (an empty delta: never valid).
 * Outputs: parent[max_nodes], state[max_nodes][R], node_prob[max_nodes]
 * (probability of the entry the node added; root: 1), returns the node count.
 * ---------------------------------------------------------------------- */
int oracle_build_draft_tree(int R, int k, const int32_t* root_state, int32_t mask_id,
                            const int32_t* topk_idx, const float* topk_prob, int W, int D,
                            int max_nodes, int32_t* parent, int32_t* state, float* node_prob) {
  int n = 1;
  parent[0] = -1;
  node_prob[0] = 1.0f;
  memcpy(state, root_state, sizeof(int32_t) * (size_t)R);
  for (int b = 1; b < max_nodes; ++b) {
    parent[b] = 0;
    node_prob[b] = 0.0f;
    memcpy(state + (size_t)b * R, root_state, sizeof(int32_t) * (size_t)R);
  }
  int* frontier = (int*)malloc(sizeof(int) * (size_t)(max_nodes > 0 ? max_nodes : 1));
  int n_front = 1;
  frontier[0] = 0;
  /* children of one level before pruning: (parent node, row, rank) */
  const int cap = (k > max_nodes ? k : max_nodes) + 1;
  int* c_par = (int*)malloc(sizeof(int) * (size_t)cap);
  int* c_row = (int*)malloc(sizeof(int) * (size_t)cap);
  int* c_rank = (int*)malloc(sizeof(int) * (size_t)cap);
  uint8_t* used = (uint8_t*)malloc((size_t)R * (size_t)k);
  for (int level = 1; level <= D && n < max_nodes && n_front > 0; ++level) {
    int n_child = 0;
    if (level == 1) {
      memset(used, 0, (size_t)R * (size_t)k);
      for (int t = 0; t < k; ++t) {  /* the k best pool entries, one scan each */
        int br = -1, bj = -1;
        for (int r = 0; r < R; ++r) {
          if (root_state[r] != mask_id) continue;
          for (int j = 0; j < k; ++j) {
            if (used[r * k + j]) continue;
            if (br < 0 || topk_prob[r * k + j] > topk_prob[br * k + bj]) { br = r; bj = j; }
          }
        }
        if (br < 0) break;
        used[br * k + bj] = 1;
        c_par[n_child] = 0; c_row[n_child] = br; c_rank[n_child] = bj; ++n_child;
      }
    } else {
      for (int f = 0; f < n_front; ++f) {
        const int32_t* ps = state + (size_t)frontier[f] * R;
        int br = -1, bj = -1;
        for (int r = 0; r < R; ++r) {
          if (ps[r] != mask_id) continue;
          for (int j = 0; j < k; ++j)
            if (br < 0 || topk_prob[r * k + j] > topk_prob[br * k + bj]) { br = r; bj = j; }
        }
        if (br < 0) continue;  /* the node is full: nothing left to speculate on */
        c_par[n_child] = frontier[f]; c_row[n_child] = br; c_rank[n_child] = bj; ++n_child;
      }
    }
    /* PruneByConfidence: stable selection of the W most probable children */
    n_front = 0;
    for (int w = 0; w < W && n < max_nodes; ++w) {
      int best = -1;
      for (int c = 0; c < n_child; ++c) {
        if (c_par[c] < 0) continue;
        if (best < 0 || topk_prob[c_row[c] * k + c_rank[c]] > topk_prob[c_row[best] * k + c_rank[best]]) best = c;
      }
      if (best < 0) break;
      const int b = n++;
      parent[b] = c_par[best];
      memcpy(state + (size_t)b * R, state + (size_t)c_par[best] * R, sizeof(int32_t) * (size_t)R);
      state[(size_t)b * R + c_row[best]] = topk_idx[c_row[best] * k + c_rank[best]];
      node_prob[b] = topk_prob[c_row[best] * k + c_rank[best]];
      frontier[n_front++] = b;
      c_par[best] = -1;
    }
  }
  free(frontier); free(c_par); free(c_row); free(c_rank); free(used);
  return n;
}
