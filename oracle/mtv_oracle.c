/*
 * TEST INFRASTRUCTURE — not part of the product.
 *
 * Plain fp64 CPU statement of what the static-tree verification path computes
 * (Section 3.1 "Multi-Head Prediction Architecture", Section 3.2 "Static
 * Implementation": Tensorization of Tree Topology, Zero-Copy Retrieval).
 * The method is exact — tree verification reaches the result of sequential
 * greedy decoding — so every function below is the plain definition written
 * out: no blocking, no online softmax, no bitmasks, no fusion.  All inputs are
 * bf16 bit patterns (uint16_t); bf16 -> double is exact.  `omp parallel for`
 * only distributes independent outputs; it never changes the arithmetic of
 * one output.
 *
 * Shares no code with the CUDA library.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may load this file's shared object.
 *
 * Pins (tests/test_oracle_*.py): heads — printed sigmoid constants, the
 *   W1=0 reduction to a plain matrix-vector product, transposition / head
 *   mix-up detectors; top-k — brute force, duplicate rows; attention — equals
 *   single-query causal attention over [prefix ; root-to-node path] computed
 *   by a library routine, closed forms for equal keys and an empty prefix;
 *   accept — brute-force sequential greedy decoding of a toy model; compaction
 *   — one-at-a-time append; LM head — one-hot hidden states that select a weight column,
 *   a hand-computed 3x4 case, planted ties, a library matrix product.  No function here is
 *   "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t x) {
    uint32_t u = (uint32_t)x << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ------------------------------------------------------------------ heads
 * Section 3.1: K parallel heads after the final layer, each an MLP with a
 * residual connection, projecting h_t to a distribution over the vocabulary.
 * One residual SiLU block then the vocabulary projection:
 *     y  = W1_k h + b1_k
 *     h' = h + y * sigmoid(y)
 *     z_k = W2_k h'
 * with no intermediate rounding.  z is [K][B][V] doubles.
 */
void mtv_ref_heads_logits(int K, int B, int H, int V,
                          const uint16_t *hidden, /* [B][H] */
                          const uint16_t *W1,     /* [K][H][H], out-feature major */
                          const uint16_t *b1,     /* [K][H] or NULL */
                          const uint16_t *W2,     /* [K][V][H] */
                          double *z)              /* [K][B][V] */
{
    for (int k = 0; k < K; ++k) {
        for (int b = 0; b < B; ++b) {
            double *hp = (double *)malloc(sizeof(double) * (size_t)H);
#pragma omp parallel for schedule(static)
            for (int o = 0; o < H; ++o) {
                double y = b1 ? bf16_to_double(b1[(size_t)k * H + o]) : 0.0;
                const uint16_t *w = W1 + ((size_t)k * H + o) * H;
                for (int i = 0; i < H; ++i)
                    y += bf16_to_double(w[i]) * bf16_to_double(hidden[(size_t)b * H + i]);
                double silu = y / (1.0 + exp(-y));
                hp[o] = bf16_to_double(hidden[(size_t)b * H + o]) + silu;
            }
#pragma omp parallel for schedule(static)
            for (int v = 0; v < V; ++v) {
                const uint16_t *w = W2 + ((size_t)k * V + v) * H;
                double acc = 0.0;
                for (int i = 0; i < H; ++i)
                    acc += bf16_to_double(w[i]) * hp[i];
                z[((size_t)k * B + b) * V + v] = acc;
            }
            free(hp);
        }
    }
}

/* ------------------------------------------------------------------ top-k
 * Candidates of one head: the k largest logits, in descending order, equal
 * logits ordered by ascending token id.  Stable ordering of (-z_v, v).
 * Also reports the smallest gap between consecutive ranks 1..k+1, which the
 * tests use to reject seeds whose ranking is decided below fp32 resolution.
 */
typedef struct { double z; int32_t v; } zv_t;
static int zv_cmp(const void *a, const void *b) {
    const zv_t *x = (const zv_t *)a, *y = (const zv_t *)b;
    if (x->z > y->z) return -1;
    if (x->z < y->z) return 1;
    return (x->v > y->v) - (x->v < y->v);
}
void mtv_ref_topk(int V, const double *z, int k, int32_t *ids, double *vals, double *min_gap)
{
    zv_t *a = (zv_t *)malloc(sizeof(zv_t) * (size_t)V);
    for (int v = 0; v < V; ++v) { a[v].z = z[v]; a[v].v = v; }
    qsort(a, (size_t)V, sizeof(zv_t), zv_cmp);
    double g = INFINITY;
    for (int r = 0; r < k; ++r) {
        ids[r] = a[r].v;
        if (vals) vals[r] = a[r].z;
        if (r + 1 < V && a[r].z - a[r + 1].z < g) g = a[r].z - a[r + 1].z;
    }
    if (min_gap) *min_gap = g;
    free(a);
}

/* -------------------------------------------------------------- attention
 * Section 3.2 / Fig. 2(b): every tree node attends to the prefix and to the
 * nodes that medusa_attn_mask [T][T] marks visible for it (its ancestors and
 * itself).  Node a's K/V live in cache slot L_b + a.  For query (b, i, h),
 * KV head g = h / (Hq/Hkv):
 *     visible = {0..L_b-1} U {L_b + a : mask[i][a] != 0}
 *     s_j = scale * <q, k_j>,  w = softmax over visible,  o = sum w_j v_j
 * Two-pass softmax in fp64.  Cache layout by element strides (sb, sh, st).
 */
static void attention_row(int T, int Hq, int Hkv, int D,
                          const uint16_t *q, const uint16_t *kc, const uint16_t *vc,
                          int64_t sb, int64_t sh, int64_t st,
                          const int32_t *seq_lens, const uint8_t *mask, double scale,
                          int b, int i, int h, double *o)
{
    int g = h / (Hq / Hkv);
    int L = seq_lens[b];
    int *vis = (int *)malloc(sizeof(int) * (size_t)(L + T));
    int n = 0;
    for (int j = 0; j < L; ++j) vis[n++] = j;
    for (int a = 0; a < T; ++a)
        if (mask[(size_t)i * T + a]) vis[n++] = L + a;
    double *s = (double *)malloc(sizeof(double) * (size_t)n);
    const uint16_t *qr = q + (((size_t)b * T + i) * Hq + h) * D;
    double m = -INFINITY;
    for (int t = 0; t < n; ++t) {
        const uint16_t *kr = kc + b * sb + g * sh + (int64_t)vis[t] * st;
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += bf16_to_double(qr[d]) * bf16_to_double(kr[d]);
        s[t] = scale * dot;
        if (s[t] > m) m = s[t];
    }
    double sum = 0.0;
    for (int t = 0; t < n; ++t) { s[t] = exp(s[t] - m); sum += s[t]; }
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    for (int t = 0; t < n; ++t) {
        const uint16_t *vr = vc + b * sb + g * sh + (int64_t)vis[t] * st;
        double w = s[t] / sum;
        for (int d = 0; d < D; ++d) o[d] += w * bf16_to_double(vr[d]);
    }
    free(s);
    free(vis);
}

void mtv_ref_tree_attention(int B, int T, int Hq, int Hkv, int D,
                            const uint16_t *q, const uint16_t *kc, const uint16_t *vc,
                            int64_t sb, int64_t sh, int64_t st,
                            const int32_t *seq_lens, const uint8_t *mask, double scale,
                            double *out /* [B][T][Hq][D] */)
{
    int n = B * T * Hq;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n; ++r) {
        int b = r / (T * Hq), i = (r / Hq) % T, h = r % Hq;
        attention_row(T, Hq, Hkv, D, q, kc, vc, sb, sh, st, seq_lens, mask, scale, b, i, h,
                      out + (size_t)r * D);
    }
}

/* The same, for a caller-chosen list of (b, i, h) triples: out is [n][D]. */
void mtv_ref_tree_attention_rows(int T, int Hq, int Hkv, int D,
                                 const uint16_t *q, const uint16_t *kc, const uint16_t *vc,
                                 int64_t sb, int64_t sh, int64_t st,
                                 const int32_t *seq_lens, const uint8_t *mask, double scale,
                                 int n, const int32_t *rows /* [n][3] */, double *out)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n; ++r)
        attention_row(T, Hq, Hkv, D, q, kc, vc, sb, sh, st, seq_lens, mask, scale,
                      rows[3 * r], rows[3 * r + 1], rows[3 * r + 2], out + (size_t)r * D);
}

/* ----------------------------------------------------------------- accept
 * Section 3.2, Zero-Copy Retrieval: the best candidate path is identified by
 * the acceptance criterion (greedy exact match, longest prefix), then the
 * final token sequence is gathered from the candidates through
 * retrieve_indices [P][K+1] (-1 padded).
 *   am[b][i]  = argmax_v logits[b][i][v]           (ties: lowest v)
 *   len_p     = number of leading j >= 1 with
 *               tree_tok[b][ri[p][j]] == am[b][ri[p][j-1]]
 *   best      = argmax_p len_p                     (ties: lowest p)
 */
void mtv_ref_node_argmax(int B, int T, int V, const uint16_t *logits, int32_t *am)
{
    int n = B * T;
#pragma omp parallel for schedule(static)
    for (int r = 0; r < n; ++r) {
        const uint16_t *row = logits + (size_t)r * V;
        int best = 0;
        double bz = bf16_to_double(row[0]);
        for (int v = 1; v < V; ++v) {
            double x = bf16_to_double(row[v]);
            if (x > bz) { bz = x; best = v; }
        }
        am[r] = best;
    }
}

void mtv_ref_tree_accept(int B, int T, int K, int P,
                         const int32_t *am,       /* [B][T] */
                         const int32_t *tree_tok, /* [B][T] */
                         const int32_t *ri,       /* [P][K+1] */
                         int32_t *accept_len, int32_t *best_path,
                         int32_t *acc_nodes /* [B][K+1] */, int32_t *acc_tok /* [B][K+1] */,
                         int32_t *next_root)
{
    for (int b = 0; b < B; ++b) {
        int best = 0, best_len = -1;
        for (int p = 0; p < P; ++p) {
            const int32_t *path = ri + (size_t)p * (K + 1);
            int len = 0;
            for (int j = 1; j <= K; ++j) {
                if (path[j] < 0) break;
                if (tree_tok[(size_t)b * T + path[j]] != am[(size_t)b * T + path[j - 1]]) break;
                len = j;
            }
            if (len > best_len) { best_len = len; best = p; }
        }
        accept_len[b] = best_len;
        best_path[b] = best;
        for (int j = 0; j <= K; ++j) {
            int node = j <= best_len ? ri[(size_t)best * (K + 1) + j] : -1;
            acc_nodes[(size_t)b * (K + 1) + j] = node;
            acc_tok[(size_t)b * (K + 1) + j] = node >= 0 ? tree_tok[(size_t)b * T + node] : -1;
        }
        next_root[b] = am[(size_t)b * T + ri[(size_t)best * (K + 1) + best_len]];
    }
}

/* ------------------------------------------------------------- compaction
 * Zero-copy retrieval applied to K/V: after acceptance the rows of the
 * accepted nodes, stored at L_b + acc_nodes[j], become rows L_b + j
 * (j = 1..accept_len); the root row (j = 0) is already in place.  Then
 * seq_len grows by accept_len + 1.  Written out of place: every source row is
 * read from the untouched copy `src`.
 * One cache of element strides (sb, sh, st); rows are D contiguous elements.
 */
void mtv_ref_kv_compact(int B, int Hkv, int D,
                        const uint16_t *src, uint16_t *dst, size_t n_elems,
                        int64_t sb, int64_t sh, int64_t st,
                        const int32_t *seq_lens, const int32_t *accept_len,
                        const int32_t *acc_nodes, int K)
{
    memcpy(dst, src, n_elems * sizeof(uint16_t));
    for (int b = 0; b < B; ++b)
        for (int g = 0; g < Hkv; ++g)
            for (int j = 1; j <= accept_len[b]; ++j) {
                int64_t from = seq_lens[b] + acc_nodes[(size_t)b * (K + 1) + j];
                int64_t to = seq_lens[b] + j;
                memcpy(dst + b * sb + g * sh + to * st, src + b * sb + g * sh + from * st,
                       (size_t)D * sizeof(uint16_t));
            }
}

/* ------------------------------------------------------ tree K/V append + RoPE
 * The step just before the tree attention (Section 3.2: tree_indices maps the flattened tree
 * nodes to their positions): node i of sequence b sits at position seq_lens[b] + depth[i] and
 * its K / V rows go to cache row seq_lens[b] + i.  Rotary embedding in the rotate-half pairing:
 * for d < D/2, angle = position * theta^(-2d/D),
 *     (x[d], x[d + D/2]) -> (x[d] cos - x[d + D/2] sin,  x[d + D/2] cos + x[d] sin).
 * q [B][T][Hq][D] and k_new, v_new [B][T][Hkv][D] are bf16; the rotated q and k come back as
 * doubles (q_out [B][T][Hq][D], k_out [B][T][Hkv][D]); V is copied unchanged by the caller.
 */
void mtv_ref_rope(int B, int T, int Hq, int Hkv, int D,
                  const uint16_t *q, const uint16_t *k_new, const int32_t *seq_lens, const int32_t *depth,
                  double theta, double *q_out, double *k_out)
{
    const int half = D / 2;
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < T; ++i) {
            const double pos = (double)seq_lens[b] + (double)depth[i];
            for (int which = 0; which < 2; ++which) {
                const int Hn = which ? Hkv : Hq;
                const uint16_t *src = which ? k_new : q;
                double *dst = which ? k_out : q_out;
                for (int h = 0; h < Hn; ++h) {
                    const size_t base = (((size_t)b * T + i) * Hn + h) * D;
                    for (int d = 0; d < half; ++d) {
                        const double ang = pos * pow(theta, -2.0 * d / D);
                        const double c = cos(ang), sn = sin(ang);
                        const double x1 = bf16_to_double(src[base + d]), x2 = bf16_to_double(src[base + d + half]);
                        dst[base + d] = x1 * c - x2 * sn;
                        dst[base + d + half] = x2 * c + x1 * sn;
                    }
                }
            }
        }
}

/* ------------------------------------------------------ LM head + per-node argmax
 * The base model's last projection as the acceptance of Section 3.2 uses it: at every tree node
 * m the most likely token  am[m] = argmax_v z[m][v],  z[m][v] = sum_h x[m][h] W[v][h]
 * (ties: lowest v).  x [M][H] and W [V][H] are bf16.  zmax[m] = z[m][am[m]]; z2[m] = the largest
 * z[m][v] over v != am[m] (-inf if V == 1), which tells a test how decisive the argmax was.
 * z_out (may be NULL) receives all logits [M][V].
 */
void mtv_ref_lm_head_argmax(int M, int H, int V, const uint16_t *x, const uint16_t *W,
                            int32_t *am, double *zmax, double *z2, double *z_out)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        int best = -1;
        double bz = 0.0, second = -INFINITY;
        for (int v = 0; v < V; ++v) {
            double z = 0.0;
            for (int h = 0; h < H; ++h)
                z += bf16_to_double(x[(size_t)m * H + h]) * bf16_to_double(W[(size_t)v * H + h]);
            if (z_out) z_out[(size_t)m * V + v] = z;
            if (best < 0) { best = v; bz = z; }
            else if (z > bz) { second = bz; bz = z; best = v; }
            else if (z > second) second = z;
        }
        am[m] = best; zmax[m] = bz; z2[m] = second;
    }
}
