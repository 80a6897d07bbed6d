// Host side of the library: static tree tensors (Section 3.2, "Tensorization of
// Tree Topology" and the retrieve_indices table of "Zero-Copy Retrieval"), the two
// tree generators, and the upload of the tables to the device.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <new>

#include "common.cuh"

namespace {

thread_local char g_err[256] = "no error";

using Tuple = std::vector<int32_t>;

struct TupleLess {
    bool operator()(const Tuple &a, const Tuple &b) const {
        if (a.size() != b.size()) return a.size() < b.size();
        return a < b;  // lexicographic
    }
};

}  // namespace

namespace mtv {
void set_last_error(const char *what, cudaError_t e) {
    snprintf(g_err, sizeof g_err, "%s: %s", what, cudaGetErrorString(e));
}
void set_last_error_text(const char *text) { snprintf(g_err, sizeof g_err, "%s", text); }
int sm_count() {
    static int n[MTV_MAX_DEVICES] = {0};
    int dev = 0, count = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MTV_MAX_DEVICES) return 148;
    if (n[dev] == 0) {
        if (cudaDeviceGetAttribute(&count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || count <= 0) count = 148;
        n[dev] = count;
    }
    return n[dev];
}
Tap g_taps[MTV_KERNEL_COUNT];
}  // namespace mtv

extern "C" int mtv_set_kernel_taps(int id, void **start, void **stop, int capacity) {
    if (id < 0 || id >= MTV_KERNEL_COUNT) return MTV_ERR_INVALID_ARG;
    mtv::Tap &t = mtv::g_taps[id];
    const bool on = start && stop && capacity > 0;
    t.start = on ? reinterpret_cast<cudaEvent_t *>(start) : nullptr;
    t.stop = on ? reinterpret_cast<cudaEvent_t *>(stop) : nullptr;
    t.cap = on ? capacity : 0;
    t.n = 0;
    return MTV_OK;
}
extern "C" int mtv_kernel_taps_used(int id) {
    return id < 0 || id >= MTV_KERNEL_COUNT ? -1 : mtv::g_taps[id].n;
}

extern "C" const char *mtv_last_error(void) { return g_err; }

extern "C" int tree_build_static(int K, int n_nodes, const int32_t *node_ranks, int upload, mtv_tree_t **out) {
    if (!out) return MTV_ERR_INVALID_ARG;
    *out = nullptr;
    if (K < 1 || n_nodes < 0 || (n_nodes > 0 && !node_ranks)) return MTV_ERR_INVALID_ARG;
    if (K > MTV_MAX_K || n_nodes + 1 > MTV_MAX_T) return MTV_ERR_UNSUPPORTED_SHAPE;

    // 1. read the tuples, order them breadth-first: (depth, rank tuple) ascending
    std::map<Tuple, int, TupleLess> index;
    index[Tuple()] = 0;
    for (int n = 0; n < n_nodes; ++n) {
        Tuple t;
        bool ended = false;
        for (int d = 0; d < K; ++d) {
            int32_t r = node_ranks[(size_t)n * K + d];
            if (r < 0) { ended = true; continue; }
            if (ended) return MTV_ERR_INVALID_ARG;  // a rank after the padding
            if (r >= MTV_MAX_TOPK) return MTV_ERR_UNSUPPORTED_SHAPE;
            t.push_back(r);
        }
        if (t.empty()) return MTV_ERR_INVALID_ARG;
        if (!index.emplace(t, 0).second) return MTV_ERR_INVALID_ARG;  // duplicate
    }
    mtv_tree *tr = new (std::nothrow) mtv_tree();
    if (!tr) return MTV_ERR_INVALID_ARG;
    const int T = (int)index.size();
    tr->T = T;
    tr->K = K;
    std::vector<Tuple> order;
    order.reserve(T);
    {
        int i = 0;
        for (auto &kv : index) { kv.second = i++; order.push_back(kv.first); }
    }
    // 2. parent / depth / rank; every parent must exist
    tr->parent.assign(T, -1);
    tr->depth.assign(T, 0);
    tr->rank.assign(T, -1);
    tr->node_ranks.assign((size_t)T * K, -1);
    for (int i = 1; i < T; ++i) {
        const Tuple &t = order[i];
        Tuple par(t.begin(), t.end() - 1);
        auto it = index.find(par);
        if (it == index.end()) { delete tr; return MTV_ERR_INVALID_ARG; }
        tr->parent[i] = it->second;
        tr->depth[i] = (int)t.size();
        tr->rank[i] = t.back();
        for (size_t d = 0; d < t.size(); ++d) tr->node_ranks[(size_t)i * K + d] = t[d];
        tr->k_d[t.size() - 1] = std::max(tr->k_d[t.size() - 1], t.back() + 1);
    }
    // 3. candidate buffer layout and tree_indices
    int off = 1;
    for (int d = 0; d < K; ++d) { tr->cand_offset[d] = off; off += tr->k_d[d]; }
    tr->C = off;
    tr->tree_indices.assign(T, 0);
    for (int i = 1; i < T; ++i) tr->tree_indices[i] = tr->cand_offset[tr->depth[i] - 1] + tr->rank[i];
    // 4. visibility: ancestor-or-self sets as bit rows and as the dense matrix
    tr->anc_words = (T + 63) / 64;
    tr->anc.assign((size_t)T * tr->anc_words, 0);
    tr->mask.assign((size_t)T * T, 0);
    for (int i = 0; i < T; ++i)
        for (int j = i; j >= 0; j = tr->parent[j]) {
            tr->anc[(size_t)i * tr->anc_words + j / 64] |= 1ull << (j % 64);
            tr->mask[(size_t)i * T + j] = 1;
        }
    // 5. one path per leaf, ascending leaf index
    std::vector<char> has_child(T, 0);
    for (int i = 1; i < T; ++i) has_child[tr->parent[i]] = 1;
    for (int i = 0; i < T; ++i) {
        if (has_child[i]) continue;
        std::vector<int32_t> path(K + 1, -1);
        for (int j = i; j >= 0; j = tr->parent[j]) path[tr->depth[j]] = j;
        tr->retrieve.insert(tr->retrieve.end(), path.begin(), path.end());
        tr->P++;
    }
    // 6. upload
    if (upload) {
        const size_t n_ti = T, n_ri = (size_t)tr->P * (K + 1), n_anc = (size_t)T * 2;
        size_t o_ti = 0, o_ri = mtv::align_up(o_ti + n_ti * 4, 16), o_anc = mtv::align_up(o_ri + n_ri * 4, 16);
        size_t o_kd = o_anc + n_anc * 8, o_co = o_kd + MTV_MAX_K * 4, o_err = o_co + MTV_MAX_K * 4, o_cnt = o_err + 16, o_dep = o_cnt + 512 * 4, total = o_dep + (size_t)T * 4;
        std::vector<unsigned char> blob(total, 0);
        memcpy(blob.data() + o_ti, tr->tree_indices.data(), n_ti * 4);
        memcpy(blob.data() + o_ri, tr->retrieve.data(), n_ri * 4);
        for (int i = 0; i < T; ++i)
            for (int w = 0; w < tr->anc_words; ++w)
                memcpy(blob.data() + o_anc + ((size_t)i * 2 + w) * 8, &tr->anc[(size_t)i * tr->anc_words + w], 8);
        memcpy(blob.data() + o_kd, tr->k_d, MTV_MAX_K * 4);
        memcpy(blob.data() + o_co, tr->cand_offset, MTV_MAX_K * 4);
        memcpy(blob.data() + o_dep, tr->depth.data(), (size_t)T * 4);
        cudaError_t e = cudaGetDevice(&tr->device);
        if (e == cudaSuccess) e = cudaMalloc(&tr->d_blob, total);
        if (e == cudaSuccess) e = cudaMemcpy(tr->d_blob, blob.data(), total, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            mtv::set_last_error("tree upload", e);
            if (tr->d_blob) cudaFree(tr->d_blob);
            delete tr;
            return MTV_ERR_CUDA;
        }
        char *base = (char *)tr->d_blob;
        tr->d_tree_indices = (const int32_t *)(base + o_ti);
        tr->d_retrieve = (const int32_t *)(base + o_ri);
        tr->d_anc = (const uint64_t *)(base + o_anc);
        tr->d_kd = (const int32_t *)(base + o_kd);
        tr->d_cand_offset = (const int32_t *)(base + o_co);
        tr->d_error = (int32_t *)(base + o_err);
        tr->d_counters = (int32_t *)(base + o_cnt);
        tr->d_depth = (const int32_t *)(base + o_dep);
        tr->on_device = true;
    }
    *out = tr;
    return MTV_OK;
}

extern "C" void tree_destroy(mtv_tree_t *tree) {
    if (!tree) return;
    if (tree->d_blob) cudaFree(tree->d_blob);
    delete tree;
}

extern "C" int mtv_device_error(const mtv_tree_t *tree, int clear, int32_t *code) {
    if (!tree || !tree->on_device || !code) return MTV_ERR_INVALID_ARG;
    MTV_CUDA_CHECK(cudaMemcpy(code, tree->d_error, sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (clear && *code != 0) {   // an aborted kernel may also have left the merge counters dirty
        MTV_CUDA_CHECK(cudaMemset(tree->d_error, 0, sizeof(int32_t)));
        MTV_CUDA_CHECK(cudaMemset(tree->d_counters, 0, 512 * sizeof(int32_t)));
    }
    return MTV_OK;
}

extern "C" int tree_query(const mtv_tree_t *t, mtv_tree_info *info) {
    if (!t || !info) return MTV_ERR_INVALID_ARG;
    memset(info, 0, sizeof *info);
    info->T = t->T; info->K = t->K; info->P = t->P; info->C = t->C;
    info->anc_words = t->anc_words;
    info->on_device = t->on_device ? 1 : 0;
    for (int d = 0; d < MTV_MAX_K; ++d) { info->k_d[d] = t->k_d[d]; info->cand_offset[d] = t->cand_offset[d]; }
    info->node_ranks = t->node_ranks.data();
    info->parent = t->parent.data();
    info->depth = t->depth.data();
    info->rank = t->rank.data();
    info->tree_indices = t->tree_indices.data();
    info->retrieve_indices = t->retrieve.data();
    info->anc = t->anc.data();
    info->medusa_attn_mask = t->mask.data();
    return MTV_OK;
}

extern "C" int tree_gen_cartesian(int K, const int32_t *topk, int capacity, int32_t *node_ranks, int *n_nodes) {
    if (K < 1 || K > MTV_MAX_K || !topk || !n_nodes) return MTV_ERR_INVALID_ARG;
    long total = 0, level = 1;
    for (int d = 0; d < K; ++d) {
        if (topk[d] < 1 || topk[d] > MTV_MAX_TOPK) return MTV_ERR_INVALID_ARG;
        level *= topk[d];
        total += level;
        if (total > 1 << 20) return MTV_ERR_UNSUPPORTED_SHAPE;
    }
    *n_nodes = (int)total;
    if (capacity < total || !node_ranks) return MTV_ERR_INVALID_ARG;
    int n = 0;
    std::vector<int32_t> t;
    // enumerate depth by depth with a mixed-radix counter
    for (int d = 1; d <= K; ++d) {
        t.assign(d, 0);
        while (true) {
            for (int j = 0; j < K; ++j) node_ranks[(size_t)n * K + j] = j < d ? t[j] : -1;
            ++n;
            int j = d - 1;
            while (j >= 0 && ++t[j] == topk[j]) t[j--] = 0;
            if (j < 0) break;
        }
    }
    return MTV_OK;
}

namespace {
// A node of the full R-ary tree with the integer form of 1/score:
// 1/score = prod(r_d + 1) * Z^depth, Z = zn/zd.  Two nodes a, b with depths
// da >= db compare as  prod_a * zn^(da-db)  vs  prod_b * zd^(da-db).
struct Scored {
    unsigned __int128 prod;
    int depth;
    Tuple t;
};
unsigned __int128 ipow(unsigned __int128 b, int e) {
    unsigned __int128 r = 1;
    while (e-- > 0) r *= b;
    return r;
}
}  // namespace

extern "C" int tree_gen_rank_prior(int K, int T_total, int R_max, int32_t *node_ranks, int *n_nodes) {
    if (K < 1 || K > 7 || R_max < 1 || R_max > MTV_MAX_TOPK || T_total < 1 || !n_nodes) return MTV_ERR_INVALID_ARG;
    // Z = sum_{r<R} 1/(r+1) as a reduced fraction zn/zd
    unsigned long long zn = 0, zd = 1;
    for (int r = 0; r < R_max; ++r) {
        zn = zn * (r + 1) + zd;
        zd = zd * (r + 1);
        unsigned long long a = zn, b = zd;
        while (b) { unsigned long long c = a % b; a = b; b = c; }
        zn /= a; zd /= a;
    }
    // the cross-multiplied comparison below must fit 128 bits
    if (K * log2((double)R_max) + (K - 1) * log2((double)(zn > zd ? zn : zd)) > 126.0) return MTV_ERR_UNSUPPORTED_SHAPE;
    std::vector<Scored> all;
    for (int d = 1; d <= K; ++d) {
        Tuple t(d, 0);
        while (true) {
            unsigned __int128 p = 1;
            for (int r : t) p *= (unsigned)(r + 1);
            all.push_back({p, d, t});
            int j = d - 1;
            while (j >= 0 && ++t[j] == R_max) t[j--] = 0;
            if (j < 0) break;
        }
    }
    const int want = T_total - 1;
    if ((size_t)want > all.size()) return MTV_ERR_INVALID_ARG;
    const unsigned __int128 ZN = zn, ZD = zd;
    auto better = [&](const Scored &a, const Scored &b) {  // a strictly before b
        unsigned __int128 lhs, rhs;  // lhs = 1/score(a) (scaled), rhs = 1/score(b) (scaled)
        if (a.depth >= b.depth) {
            lhs = a.prod * ipow(ZN, a.depth - b.depth);
            rhs = b.prod * ipow(ZD, a.depth - b.depth);
        } else {
            lhs = a.prod * ipow(ZD, b.depth - a.depth);
            rhs = b.prod * ipow(ZN, b.depth - a.depth);
        }
        if (lhs != rhs) return lhs < rhs;          // higher score first
        if (a.depth != b.depth) return a.depth < b.depth;
        return a.t < b.t;
    };
    std::sort(all.begin(), all.end(), better);
    *n_nodes = want;
    if (!node_ranks && want > 0) return MTV_ERR_INVALID_ARG;
    for (int n = 0; n < want; ++n)
        for (int j = 0; j < K; ++j) node_ranks[(size_t)n * K + j] = j < all[n].depth ? all[n].t[j] : -1;
    return MTV_OK;
}
