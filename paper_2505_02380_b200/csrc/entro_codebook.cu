// entro_build_codebook: Huffman code lengths by pair merging (Section 3, "Huffman weight
// encoding") with two queues, then canonical code assignment.  Host only.
#include <algorithm>
#include <cstring>

#include "entro_internal.h"

namespace {

struct Node {
    uint64_t weight;
    int parent;
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

    // Canonical codes: count the codes of each length, derive the first code of each
    // length, then hand codes out in symbol order.
    uint32_t per_len[ENTRO_MAX_CODE_LEN + 2] = {0};
    for (int k = 0; k < nsym; ++k) per_len[cb->len[k]]++;
    per_len[0] = 0;
    uint64_t next_code[ENTRO_MAX_CODE_LEN + 2] = {0};
    uint64_t code = 0;
    for (int l = 1; l <= max_len; ++l) {
        code = (code + per_len[l - 1]) << 1;
        next_code[l] = code;
    }
    for (int k = 0; k < nsym; ++k)
        if (cb->len[k]) cb->code[k] = (uint32_t)next_code[cb->len[k]]++;
    return ENTRO_OK;
}
