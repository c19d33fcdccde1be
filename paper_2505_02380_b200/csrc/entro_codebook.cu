// entro_build_codebook: Huffman code lengths by pair merging (Section 3, "Huffman weight
// encoding") with two queues, then canonical code assignment.  entro_build_codebook_limited:
// the same under a cap on the code length (package-merge).  Host only.
#include <algorithm>
#include <cstring>
#include <vector>

#include "entro_internal.h"

namespace {

struct Node {
    uint64_t weight;
    int parent;
};

// Canonical codes from the lengths: count the codes of each length, derive the first code
// of each length, then hand codes out in symbol order.  (Takes the two arrays rather than the
// codebook struct: g++ 13's interprocedural mod/ref analysis dropped the stores made through
// a pointer to the typedef'd unnamed struct.)
void assign_canonical_codes(const uint8_t* len, uint32_t* code_out, int nsym, int max_len)
{
    uint32_t per_len[ENTRO_MAX_CODE_LEN + 2] = {0};
    for (int k = 0; k < nsym; ++k) per_len[len[k]]++;
    per_len[0] = 0;
    uint64_t next_code[ENTRO_MAX_CODE_LEN + 2] = {0};
    uint64_t code = 0;
    for (int l = 1; l <= max_len; ++l) {
        code = (code + per_len[l - 1]) << 1;
        next_code[l] = code;
    }
    for (int k = 0; k < nsym; ++k)
        if (len[k]) code_out[k] = (uint32_t)next_code[len[k]]++;
}

// One entry of a level's list in the package-merge construction: a leaf, or a package of two
// entries of the level below (the deeper one).
struct Entry {
    uint64_t weight;
    int leaf;        // index into the sorted leaves, or -1
    int left, right; // package: positions in the deeper level's list
};

}  // namespace

extern "C" entro_status entro_build_codebook(const uint64_t* counts, int nsym, entro_codebook* cb)
{
    if (!counts || !cb || nsym < 1 || nsym > ENTRO_MAX_SYMBOLS) return ENTRO_ERR_INVALID_ARG;
    std::memset(cb, 0, sizeof(*cb));
    cb->nsym = nsym;

    // Leaves in ascending (count, symbol) order: queue A.
    int leaf_sym[ENTRO_MAX_SYMBOLS];
    int n_leaves = 0;
    for (int k = 0; k < nsym; ++k)
        if (counts[k]) leaf_sym[n_leaves++] = k;
    if (n_leaves == 0) return ENTRO_ERR_INVALID_ARG;
    if (n_leaves == 1) {
        cb->len[leaf_sym[0]] = 1;
        cb->max_len = 1;
        return ENTRO_OK;  // code 0
    }
    std::stable_sort(leaf_sym, leaf_sym + n_leaves,
                     [&](int a, int b) { return counts[a] < counts[b]; });  // stable: symbol order kept

    // nodes[0 .. n_leaves) are the sorted leaves, nodes[n_leaves ..) internal nodes in
    // creation order: queue B.  Internal weights never decrease, so B stays sorted.
    Node nodes[2 * ENTRO_MAX_SYMBOLS];
    for (int i = 0; i < n_leaves; ++i) nodes[i] = {counts[leaf_sym[i]], -1};
    int a = 0, b = n_leaves, end = n_leaves;
    auto take = [&]() {
        // smaller front; on equal weight the leaf goes first
        if (a < n_leaves && (b >= end || nodes[a].weight <= nodes[b].weight)) return a++;
        return b++;
    };
    for (int merges = 0; merges < n_leaves - 1; ++merges) {
        int x = take();
        int y = take();
        nodes[end] = {nodes[x].weight + nodes[y].weight, -1};
        nodes[x].parent = end;
        nodes[y].parent = end;
        ++end;
    }
    int max_len = 0;
    for (int i = 0; i < n_leaves; ++i) {
        int depth = 0;
        for (int j = i; nodes[j].parent >= 0; j = nodes[j].parent) ++depth;
        if (depth > ENTRO_MAX_CODE_LEN) {
            std::memset(cb, 0, sizeof(*cb));
            return ENTRO_ERR_CODE_TOO_LONG;
        }
        cb->len[leaf_sym[i]] = (uint8_t)depth;
        max_len = std::max(max_len, depth);
    }
    cb->max_len = max_len;

    assign_canonical_codes(cb->len, cb->code, nsym, max_len);
    return ENTRO_OK;
}

extern "C" entro_status entro_build_codebook_limited(const uint64_t* counts, int nsym, int max_len, entro_codebook* cb)
{
    if (!counts || !cb || nsym < 1 || nsym > ENTRO_MAX_SYMBOLS || max_len < 1 || max_len > ENTRO_MAX_CODE_LEN)
        return ENTRO_ERR_INVALID_ARG;
    std::memset(cb, 0, sizeof(*cb));
    cb->nsym = nsym;
    std::vector<int> leaf_sym;
    for (int k = 0; k < nsym; ++k)
        if (counts[k]) leaf_sym.push_back(k);
    const int n = (int)leaf_sym.size();
    if (n == 0) return ENTRO_ERR_INVALID_ARG;
    if (n == 1) {
        cb->len[leaf_sym[0]] = 1;
        cb->max_len = 1;
        return ENTRO_OK;
    }
    if (max_len < 31 && (1u << max_len) < (unsigned)n) return ENTRO_ERR_CODE_TOO_LONG;
    std::stable_sort(leaf_sym.begin(), leaf_sym.end(), [&](int a, int b) { return counts[a] < counts[b]; });

    // lists[d] is the list of level max_len - d: lists[0] the deepest (leaves only)
    std::vector<std::vector<Entry>> lists(max_len);
    for (int d = 0; d < max_len; ++d) {
        std::vector<Entry>& cur = lists[d];
        const std::vector<Entry>* below = d ? &lists[d - 1] : nullptr;
        const size_t npk = below ? below->size() / 2 : 0;
        size_t a = 0, b = 0;
        while (a < (size_t)n || b < npk) {
            const uint64_t wl = a < (size_t)n ? counts[leaf_sym[a]] : 0;
            const uint64_t wp = b < npk ? (*below)[2 * b].weight + (*below)[2 * b + 1].weight : 0;
            // the lighter one next; a leaf before a package of equal weight
            if (b >= npk || (a < (size_t)n && wl <= wp)) {
                cur.push_back({wl, (int)a, -1, -1});
                ++a;
            } else {
                cur.push_back({wp, -1, (int)(2 * b), (int)(2 * b + 1)});
                ++b;
            }
        }
    }
    const std::vector<Entry>& top = lists[max_len - 1];
    const size_t need = 2 * (size_t)(n - 1);
    if (top.size() < need) return ENTRO_ERR_CODE_TOO_LONG;
    // every leaf reached from one of the first 2(n - 1) entries of level 1 adds one bit
    std::vector<uint32_t> depth(n, 0);
    std::vector<std::pair<int, int>> stack;   // (list index, position)
    for (size_t i = 0; i < need; ++i) {
        stack.push_back({max_len - 1, (int)i});
        while (!stack.empty()) {
            auto [d, pos] = stack.back();
            stack.pop_back();
            const Entry& e = lists[d][pos];
            if (e.leaf >= 0) depth[e.leaf]++;
            else {
                stack.push_back({d - 1, e.left});
                stack.push_back({d - 1, e.right});
            }
        }
    }
    int longest = 0;
    for (int i = 0; i < n; ++i) {
        cb->len[leaf_sym[i]] = (uint8_t)depth[i];
        longest = std::max(longest, (int)depth[i]);
    }
    cb->max_len = longest;
    assign_canonical_codes(cb->len, cb->code, nsym, longest);
    return ENTRO_OK;
}
