// Catalog C_A, eligibility, feature schema F_A and plan table Pi_A with the online selection of
// Algorithm 2 (paper Section 4.4 and Section 5.2).  Host code only.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <mutex>
#include <string>
#include <vector>

#include "bsa_common.h"

namespace bsa {

// ---------------------------------------------------------------------------------------------
// catalog: every entry is a precompiled kernel + organisation; plan_id == index
// ---------------------------------------------------------------------------------------------
static const bsa_plan_desc_t kCatalog[] = {
    //  id  T_Q  T_KV stages tau pmax order                       kernel name
    {0, 128, 128, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 0, "q128k128"},
    {1, 128, 64, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 0, "q128k64"},
    {2, 128, 128, 0, 4, 8, BSA_ORDER_HEAD_MAJOR_LPT, 0, "q128k128_split4x8"},
    {3, 128, 64, 0, 8, 8, BSA_ORDER_HEAD_MAJOR_LPT, 0, "q128k64_split8x8"},
    {4, 128, 128, 0, 0, 1, BSA_ORDER_GLOBAL_LPT, 0, "q128k128_global"},
    {5, 128, 64, 0, 0, 1, BSA_ORDER_GLOBAL_LPT, 0, "q128k64_global"},
    {6, 128, 128, 2, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 0, "q128k128_s2"},
    {7, 128, 64, 3, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 0, "q128k64_s3"},
    {8, 128, 128, 0, 16, 4, BSA_ORDER_GLOBAL_LPT, 0, "q128k128_split16x4_global"},
    {9, 128, 64, 0, 2, 16, BSA_ORDER_HEAD_MAJOR_LPT, 0, "q128k64_split2x16"},
    // two 128-row Q tiles per CTA sharing one K/V ring, two softmax warpgroups
    {10, 256, 128, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 1, "q256k128"},
    {11, 256, 64, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 1, "q256k64"},
    {12, 256, 128, 0, 4, 8, BSA_ORDER_HEAD_MAJOR_LPT, 1, "q256k128_split4x8"},
    {13, 256, 128, 0, 0, 1, BSA_ORDER_GLOBAL_LPT, 1, "q256k128_global"},
    // one 128-row Q tile per CTA, two softmax threads per query row (column halves)
    {14, 128, 128, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 2, "q128k128_cs"},
    {15, 128, 64, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 2, "q128k64_cs"},
    {16, 128, 128, 0, 4, 8, BSA_ORDER_HEAD_MAJOR_LPT, 2, "q128k128_cs_split4x8"},
    {17, 128, 128, 0, 0, 1, BSA_ORDER_GLOBAL_LPT, 2, "q128k128_cs_global"},
    // one 128-row Q tile per CTA, separate issuing threads for Q K^T and P V
    {18, 128, 128, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 3, "q128k128_di"},
    {19, 128, 64, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 3, "q128k64_di"},
    {20, 128, 128, 0, 4, 8, BSA_ORDER_HEAD_MAJOR_LPT, 3, "q128k128_di_split4x8"},
    {21, 128, 128, 0, 0, 1, BSA_ORDER_GLOBAL_LPT, 3, "q128k128_di_global"},
    // one 128-row Q tile per CTA, two softmax warpgroups on alternate KV tiles, shared reference maximum
    {22, 128, 128, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 4, "q128k128_pp"},
    {23, 128, 64, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 4, "q128k64_pp"},
    {24, 128, 128, 0, 4, 8, BSA_ORDER_HEAD_MAJOR_LPT, 4, "q128k128_pp_split4x8"},
    {25, 128, 128, 0, 0, 1, BSA_ORDER_GLOBAL_LPT, 4, "q128k128_pp_global"},
    {26, 128, 64, 0, 0, 1, BSA_ORDER_GLOBAL_LPT, 4, "q128k64_pp_global"},
    {27, 128, 64, 0, 4, 8, BSA_ORDER_HEAD_MAJOR_LPT, 4, "q128k64_pp_split4x8"},
    {28, 128, 64, 0, 2, 16, BSA_ORDER_HEAD_MAJOR_LPT, 4, "q128k64_pp_split2x16"},
    // work items in row-major order, not sorted by length: the baseline of the task-organisation ablation (Section 4.3)
    {29, 128, 128, 0, 0, 1, BSA_ORDER_NATURAL, 4, "q128k128_pp_natural"},
    // longest first by half-octave length bucket, row-major inside a bucket (balance without giving up the K/V
    // tiles that neighbouring Q tiles share)
    {30, 128, 128, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_BUCKETS, 4, "q128k128_pp_hb"},
    {31, 128, 128, 0, 0, 1, BSA_ORDER_GLOBAL_BUCKETS, 4, "q128k128_pp_gb"},
    {32, 128, 64, 0, 0, 1, BSA_ORDER_NATURAL, 4, "q128k64_pp_natural"},
    {33, 128, 64, 0, 0, 1, BSA_ORDER_GLOBAL_BUCKETS, 4, "q128k64_pp_gb"},
    // 16-row Q tiles, one warp each, on the register-level tensor instruction (mma.sync): logical blocks of up to 64
    // rows keep their own KV lists instead of being Coarsened onto 128 rows
    {34, 16, 64, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 5, "q16k64_rb"},
    {35, 16, 32, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 5, "q16k32_rb"},
    {36, 16, 16, 0, 0, 1, BSA_ORDER_HEAD_MAJOR_LPT, 5, "q16k16_rb"},
    {37, 16, 64, 0, 0, 1, BSA_ORDER_NATURAL, 5, "q16k64_rb_natural"},
    {38, 16, 32, 0, 0, 1, BSA_ORDER_NATURAL, 5, "q16k32_rb_natural"},
};
static const int kCatalogSize = (int)(sizeof(kCatalog) / sizeof(kCatalog[0]));
static const int64_t kDefaultWorkspace = 2ll << 30;
static const size_t kPlannerSmemLimit = 200 * 1024;

static bool pow2_in(int v, int lo, int hi) { return v >= lo && v <= hi && (v & (v - 1)) == 0; }

const bsa_plan_desc_t* catalog_entry(int plan_id) {
    if (plan_id < 0 || plan_id >= kCatalogSize) return nullptr;
    return &kCatalog[plan_id];
}

int ilog2(int v) {
    int l = 0;
    while ((1 << l) < v) ++l;
    return l;
}

bool make_geom(const bsa_plan_desc_t& P, int B_Q, int B_KV, int64_t N, int64_t N_kv, int heads, MapGeom* g) {
    g->H = heads;
    g->N = N;
    g->N_kv = N_kv;
    g->B_Q = B_Q;
    g->B_KV = B_KV;
    g->T_Q = P.T_Q;
    g->T_KV = P.T_KV;
    g->slots = P.T_Q >= kTQ ? P.T_Q / kTQ : 1;                 // 128-row MMA slots (one for the 16-row tiles)
    g->sQ128 = (B_Q < kTQ && P.T_Q >= kTQ) ? kTQ / B_Q : 1;    // logical rows per slot where the slot is Coarsened
    g->nQb = (int)((N + B_Q - 1) / B_Q);
    g->nKb = (int)((N_kv + B_KV - 1) / B_KV);
    g->nQt = (int)((N + P.T_Q - 1) / P.T_Q);
    g->nKt = (int)((N_kv + P.T_KV - 1) / P.T_KV);
    g->sQ = B_Q < P.T_Q ? P.T_Q / B_Q : 1;
    g->rq = B_Q > P.T_Q ? B_Q / P.T_Q : 1;
    g->sK = B_KV < P.T_KV ? P.T_KV / B_KV : 1;
    g->rk = B_KV > P.T_KV ? B_KV / P.T_KV : 1;
    g->lgBQ = ilog2(B_Q);
    g->lgBKV = ilog2(B_KV);
    g->lgSK = ilog2(g->sK);
    return true;
}

int64_t plan_workspace_bytes(const bsa_plan_desc_t& P, int64_t N, int heads, int d) {
    if (P.split_pmax <= 1) return 0;
    const int64_t nQt = (N + P.T_Q - 1) / P.T_Q;
    return (int64_t)heads * nQt * P.split_pmax * P.T_Q * (int64_t)(d + 1) * 4;
}

// Eligible(P, R), Section 4.4: logical geometry, tensor properties, metadata format, workspace.
bool plan_eligible(int plan_id, int B_Q, int B_KV, int64_t N, int heads, int d, int64_t max_ws, int64_t N_kv = 0,
                   int dtype = BSA_DTYPE_BF16) {
    const bsa_plan_desc_t* P = catalog_entry(plan_id);
    if (!P) return false;
    if (dtype != BSA_DTYPE_BF16 && dtype != BSA_DTYPE_FP16) return false;
    // tensor property: the paired and the column-split kernels are not instantiated for half tensors
    if (dtype == BSA_DTYPE_FP16 && (P->kernel == 1 || P->kernel == 2)) return false;
    if (P->kernel == kKernelRowBlock) {
        // 16-row tiles: for logical blocks of up to 64 rows (on larger ones the 128-row tile wastes nothing that this
        // kernel could win back), KV tiles no wider than the logical block (no membership masks in this kernel) and
        // no larger than a warp's staging buffer, no Split-K
        if (B_Q > 64 || B_KV < P->T_KV || P->T_KV > rb_max_chunk(d) || P->split_pmax > 1) return false;
    }
    if (!(d == 64 || d == 128 || d == 256)) return false;
    if (!pow2_in(B_Q, 16, 256) || !pow2_in(B_KV, 16, 256)) return false;
    if (N <= 0 || heads <= 0 || N > (1ll << 30)) return false;
    MapGeom g;
    if (N_kv <= 0) N_kv = N;
    if (N_kv > (1ll << 30)) return false;
    make_geom(*P, B_Q, B_KV, N, N_kv, heads, &g);
    if (g.sQ128 * g.sK > 64) return false;  // one 64-bit membership word per 128-row slot
    if (P->split_pmax > 32) return false;   // the merge kernel keeps up to 32 partial LSEs in registers
    const int max_st = attention_max_stages(d, P->T_KV, P->kernel);
    if (max_st < 2) return false;
    if (P->stages > max_st) return false;
    if ((size_t)g.nKt * 8 * g.slots > kPlannerSmemLimit) return false;
    if (organize_smem_bytes(g, P->order, P->split_pmax) > kPlannerSmemLimit) return false;
    if ((int64_t)heads * g.nQt * (P->split_pmax < 1 ? 1 : P->split_pmax) >= (1ll << 31)) return false;
    if (max_ws <= 0) max_ws = kDefaultWorkspace;
    if (plan_workspace_bytes(*P, N, heads, d) > max_ws) return false;
    return true;
}

int base_plan(int B_Q, int B_KV, int d) {
    (void)B_Q;
    (void)B_KV;
    if (d == 256) return 19;  // q128k64_di: the kernels with P in place over S are the ones that hold a 256-column O
    return 22;  // q128k128_pp: eligible for every supported geometry (membership <= 64 bits), no workspace
}

uint64_t catalog_hash() {
    uint64_t h = 1469598103934665603ull;
    const unsigned char* p = reinterpret_cast<const unsigned char*>(kCatalog);
    for (size_t i = 0; i < sizeof(kCatalog); ++i) {
        h ^= p[i];
        h *= 1099511628211ull;
    }
    return h;
}

// ---------------------------------------------------------------------------------------------
// feature schema F_A: fixed bucket edges (Section 5.1: "predefined intervals")
// ---------------------------------------------------------------------------------------------
static const double kDensityEdges[] = {0.02, 0.05, 0.08, 0.15, 0.25, 0.45};
static const double kSkewEdges[] = {1.5, 3.0, 6.0};
static const double kRunCovEdges[] = {0.5};

static int bucket_of(double v, const double* edges, int n) {
    int b = 0;
    while (b < n && v >= edges[b]) ++b;
    return b;
}

void lut_buckets(int64_t N, double density, double skew, double run_cov, int32_t out[4]) {
    int nb = 0;
    while ((1ll << (nb + 1)) <= N) ++nb;  // floor(log2 N)
    out[0] = nb;
    out[1] = bucket_of(density, kDensityEdges, 6);
    out[2] = bucket_of(skew, kSkewEdges, 3);
    out[3] = bucket_of(run_cov, kRunCovEdges, 1);
}

// ---------------------------------------------------------------------------------------------
// plan table Pi_A
// ---------------------------------------------------------------------------------------------
struct RegimeKey {
    int B_Q, B_KV, d;      // request key k_A(R) (architecture and dtype are fixed: sm_100a, bf16)
    int nb, hb;            // bucketed request dimensions u_A(R): floor(log2 N), head bucket
    int db, sb, rb;        // bucketed mask statistics s_A(M)
    bool operator<(const RegimeKey& o) const {
        return memcmp(this, &o, sizeof(RegimeKey)) < 0;
    }
};
static std::map<RegimeKey, std::vector<int>> g_table;
static std::mutex g_mu;

// Learned second-stage partition (Section 5.1: "thresholds learned by a decision tree, whose leaves define the finer
// partitions"): one binary tree per request key over the continuous request features
//   0: log2 N    1: heads    2: active-block density    3: row-nnz skew    4: active-block-run coverage.
// An inner node sends a request left when feature < threshold; a leaf holds a ranking.  Lookup order: the request's
// fixed-edge regime if the table has it, else the leaf of its key's tree, else the key's base plan.  (Leaving each
// mask source out of the corpus in turn, this order gave a geometric-mean regret of 1.026 against 1.030 for the trees
// alone and 1.29 for the regimes alone, whose buckets a request from an unseen source hits only 22 % of the time.)
struct TreeNode {
    int feature;        // -1: leaf
    double threshold;
    int left, right;
    std::vector<int> ranked;
};
struct TreeKey {
    int B_Q, B_KV, d;
    bool operator<(const TreeKey& o) const { return memcmp(this, &o, sizeof(TreeKey)) < 0; }
};
static std::map<TreeKey, std::vector<TreeNode>> g_trees;
constexpr int kTreeFeatures = 5;
constexpr int kTreeMaxNodes = 4096;

// Leaf of the key's tree these features fall into, or -1 (no tree for the key, or a malformed one).
static int tree_leaf(const std::vector<TreeNode>& t, const double f[kTreeFeatures]) {
    int n = 0;
    for (int steps = 0; steps < kTreeMaxNodes; ++steps) {
        if (n < 0 || n >= (int)t.size()) return -1;
        const TreeNode& nd = t[n];
        if (nd.feature < 0) return n;
        n = (f[nd.feature] < nd.threshold) ? nd.left : nd.right;
    }
    return -1;
}
static int g_force_plan = -1;

static int head_bucket(int heads) { return heads <= 4 ? 0 : (heads <= 16 ? 1 : 2); }

void lut_clear() {
    std::lock_guard<std::mutex> lk(g_mu);
    g_table.clear();
    g_trees.clear();
}

int lut_num_trees() {
    std::lock_guard<std::mutex> lk(g_mu);
    return (int)g_trees.size();
}

int lut_num_regimes() {
    std::lock_guard<std::mutex> lk(g_mu);
    return (int)g_table.size();
}

// File format (text, one record per line):
//   BSA_LUT 1 | 2
//   catalog <hex hash>
//   gpu <free text>
//   regime B_Q B_KV d nb hb db sb rb : id id id ...
//   (version 2 only) tree B_Q B_KV d <number of nodes>, followed by that many lines, node 0 the root:
//     node <index> split <feature> <threshold> <left> <right>
//     node <index> leaf : id id id ...
bsa_status_t lut_load(const char* path) {
    lut_clear();
    if (!path) return BSA_ERR_INVALID_ARG;
    FILE* f = fopen(path, "r");
    if (!f) return BSA_ERR_LUT;
    char line[1024];
    bool header = false, hash_ok = false;
    int version = 0;
    std::map<RegimeKey, std::vector<int>> table;
    std::map<TreeKey, std::vector<TreeNode>> trees;
    std::vector<TreeNode>* cur_tree = nullptr;  // tree whose node lines are being read
    int nodes_left = 0;
    bsa_status_t st = BSA_OK;
    auto parse_ids = [&](const char* q, std::vector<int>* ids) {
        char* end = nullptr;
        while (true) {
            long v = strtol(q, &end, 10);
            if (end == q) break;
            if (v < 0 || v >= kCatalogSize) return false;
            ids->push_back((int)v);
            q = end;
        }
        return !ids->empty();
    };
    while (fgets(line, sizeof line, f)) {
        if (line[0] == '#' || line[0] == '\n') continue;
        if (nodes_left > 0 && strncmp(line, "node", 4)) { st = BSA_ERR_LUT; break; }  // a tree's nodes follow its header
        if (!strncmp(line, "BSA_LUT", 7)) {
            if (sscanf(line + 7, "%d", &version) != 1 || (version != 1 && version != 2)) { st = BSA_ERR_LUT; break; }
            header = true;
        } else if (!strncmp(line, "tree", 4)) {
            TreeKey k;
            memset(&k, 0, sizeof k);
            int n = 0;
            if (version != 2 || sscanf(line + 4, "%d %d %d %d", &k.B_Q, &k.B_KV, &k.d, &n) != 4 || n < 1 || n > kTreeMaxNodes ||
                trees.count(k)) { st = BSA_ERR_LUT; break; }
            cur_tree = &trees[k];
            cur_tree->assign((size_t)n, TreeNode{-2, 0.0, -1, -1, {}});  // -2: not read yet
            nodes_left = n;
        } else if (!strncmp(line, "node", 4)) {
            int idx = -1, used = 0;
            if (!cur_tree || nodes_left <= 0 || sscanf(line + 4, "%d %n", &idx, &used) != 1 || idx < 0 ||
                idx >= (int)cur_tree->size() || (*cur_tree)[idx].feature != -2) { st = BSA_ERR_LUT; break; }
            TreeNode& nd = (*cur_tree)[idx];
            const char* rest = line + 4 + used;
            if (!strncmp(rest, "split", 5)) {
                if (sscanf(rest + 5, "%d %lf %d %d", &nd.feature, &nd.threshold, &nd.left, &nd.right) != 4 || nd.feature < 0 ||
                    nd.feature >= kTreeFeatures || nd.left <= idx || nd.right <= idx || nd.left >= (int)cur_tree->size() ||
                    nd.right >= (int)cur_tree->size()) { st = BSA_ERR_LUT; break; }  // children after parents: no cycles
            } else if (!strncmp(rest, "leaf", 4)) {
                const char* colon = strchr(rest, ':');
                nd.feature = -1;
                if (!colon || !parse_ids(colon + 1, &nd.ranked)) { st = BSA_ERR_LUT; break; }
            } else { st = BSA_ERR_LUT; break; }
            --nodes_left;
        } else if (!strncmp(line, "catalog", 7)) {
            unsigned long long hsh = 0;
            if (sscanf(line + 7, "%llx", &hsh) != 1 || hsh != catalog_hash()) { st = BSA_ERR_LUT; break; }
            hash_ok = true;
        } else if (!strncmp(line, "gpu", 3)) {
            continue;
        } else if (!strncmp(line, "regime", 6)) {
            RegimeKey k;
            memset(&k, 0, sizeof k);
            int used = 0;
            if (sscanf(line + 6, "%d %d %d %d %d %d %d %d :%n", &k.B_Q, &k.B_KV, &k.d, &k.nb, &k.hb, &k.db, &k.sb, &k.rb,
                       &used) != 8 || used == 0) { st = BSA_ERR_LUT; break; }
            std::vector<int> ids;
            if (!parse_ids(line + 6 + used, &ids)) { st = BSA_ERR_LUT; break; }
            table[k] = ids;
        } else {
            st = BSA_ERR_LUT;
            break;
        }
    }
    fclose(f);
    if (st == BSA_OK && (!(header && hash_ok) || nodes_left != 0)) st = BSA_ERR_LUT;
    if (st != BSA_OK) return st;
    std::lock_guard<std::mutex> lk(g_mu);
    g_table.swap(table);
    g_trees.swap(trees);
    return BSA_OK;
}

void set_force_plan(int id) { g_force_plan = id; }
int get_force_plan() { return g_force_plan; }

// Algorithm 2, lines 6-19: z = <k, u, s>; r = rho(z); ranked list or base plan; first eligible.
int lut_select(int B_Q, int B_KV, int64_t N, int heads, int d, double density, double run_cov, double skew,
               int64_t max_ws, int* hit_out, int32_t buckets_out[4], int64_t N_kv = 0, int dtype = BSA_DTYPE_BF16) {
    int32_t b[4];
    lut_buckets(N, density, skew, run_cov, b);
    if (buckets_out) memcpy(buckets_out, b, sizeof b);
    RegimeKey k;
    memset(&k, 0, sizeof k);
    k.B_Q = B_Q; k.B_KV = B_KV; k.d = d;
    k.nb = b[0]; k.hb = head_bucket(heads);
    k.db = b[1]; k.sb = b[2]; k.rb = b[3];
    std::vector<int> ranked;
    bool hit = false;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        // 1. the fixed-edge regime of the request, if the corpus had cases in it (the finest partition)
        auto it = g_table.find(k);
        if (it != g_table.end()) {
            ranked = it->second;
            hit = true;
        }
        // 2. else the leaf of the key's learned partition: requests between the corpus's grid points
        if (!hit) {
            TreeKey tk;
            memset(&tk, 0, sizeof tk);
            tk.B_Q = B_Q; tk.B_KV = B_KV; tk.d = d;
            auto tt = g_trees.find(tk);
            if (tt != g_trees.end()) {
                const double f[kTreeFeatures] = {log2((double)(N > 0 ? N : 1)), (double)heads, density, skew, run_cov};
                const int leaf = tree_leaf(tt->second, f);
                if (leaf >= 0) {
                    ranked = tt->second[leaf].ranked;
                    hit = true;
                    if (buckets_out) buckets_out[3] = b[3] | ((leaf + 1) << 8);  // leaf index + 1 above the run-coverage bucket
                }
            }
        }
    }
    if (!hit) ranked.push_back(base_plan(B_Q, B_KV, d));
    if (hit_out) *hit_out = hit ? 1 : 0;
    for (int id : ranked)
        if (plan_eligible(id, B_Q, B_KV, N, heads, d, max_ws, N_kv, dtype)) return id;
    return -1;
}

int lut_head_bucket(int heads) { return head_bucket(heads); }
int catalog_size() { return kCatalogSize; }

}  // namespace bsa
