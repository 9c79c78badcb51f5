// Trie-based prefix index (Sec. 7.3 of the paper): insert / best-match lookup / evict over stored
// session prefixes, pruned at nodes whose path probability is below epsilon.  Host-side only; every
// operation walks one root-to-node path, O(length) map steps.  The batched device-side counterpart
// of the lookup is plc_prefix_dedup.
#include <cmath>
#include <map>
#include <new>
#include <unordered_map>
#include <vector>

#include "plc.h"

struct plc_trie {
    struct Node {
        int parent = -1;
        int token = 0;
        int refs = 0;                       // stored prefixes whose path passes through this node
        double bits = 0.0;                  // -log2 P(prefix ending here)
        std::map<int, int> children;        // token -> node, ordered
        std::map<int, int> terminals;       // ids of stored prefixes that end here (value unused)
    };
    std::vector<Node> nodes;
    std::vector<int> free_list;
    std::unordered_map<int, int> end_of;    // id -> node where the stored prefix ends
    double max_bits = INFINITY;
    long long live = 0;

    int alloc() {
        if (!free_list.empty()) { int i = free_list.back(); free_list.pop_back(); nodes[i] = Node(); return i; }
        nodes.emplace_back();
        return (int)nodes.size() - 1;
    }
};

extern "C" {

plc_status plc_trie_create(plc_trie** out, float epsilon) {
    if (!out || !(epsilon >= 0.0f) || epsilon > 1.0f) return PLC_E_INVALID;
    plc_trie* t = new (std::nothrow) plc_trie();
    if (!t) return PLC_E_CUDA;
    t->nodes.emplace_back();                // root
    if (epsilon > 0.0f) t->max_bits = -std::log2((double)epsilon);
    *out = t;
    return PLC_OK;
}

plc_status plc_trie_destroy(plc_trie* t) {
    if (!t) return PLC_E_INVALID;
    delete t;
    return PLC_OK;
}

plc_status plc_trie_insert(plc_trie* t, int32_t id, const int32_t* tokens, const float* logp2, int32_t len, int32_t* stored_len) {
    if (!t || len < 0 || (len > 0 && (!tokens || !logp2))) return PLC_E_INVALID;
    if (t->end_of.count(id)) return PLC_E_STATE;
    int cur = 0, kept = 0;
    double bits = 0.0;
    t->nodes[0].refs++;
    for (int i = 0; i < len; ++i) {
        bits -= (double)logp2[i];
        if (bits > t->max_bits) break;       // this node would have probability below epsilon
        auto it = t->nodes[cur].children.find(tokens[i]);
        int nxt;
        if (it == t->nodes[cur].children.end()) {
            nxt = t->alloc();
            t->nodes[nxt].parent = cur; t->nodes[nxt].token = tokens[i]; t->nodes[nxt].bits = bits;
            t->nodes[cur].children[tokens[i]] = nxt;
            t->live++;
        } else {
            nxt = it->second;
        }
        t->nodes[nxt].refs++;
        cur = nxt; ++kept;
    }
    t->nodes[cur].terminals[id] = 1;
    t->end_of[id] = cur;
    if (stored_len) *stored_len = kept;
    return PLC_OK;
}

plc_status plc_trie_best_match(const plc_trie* t, const int32_t* tokens, int32_t len, int32_t* id, int32_t* lcp, float* dT) {
    if (!t || len < 0 || (len > 0 && !tokens) || !id || !lcp || !dT) return PLC_E_INVALID;
    *id = -1; *lcp = 0; *dT = 0.0f;
    if (t->end_of.empty()) return PLC_OK;
    int cur = 0, m = 0;
    while (m < len) {
        auto it = t->nodes[cur].children.find(tokens[m]);
        if (it == t->nodes[cur].children.end()) break;
        cur = it->second; ++m;
    }
    *lcp = m;
    *dT = (float)t->nodes[cur].bits;
    // deepest stored ancestor reached; name one stored prefix below it: the smallest continuation
    int u = cur;
    while (t->nodes[u].terminals.empty()) u = t->nodes[u].children.begin()->second;
    *id = t->nodes[u].terminals.begin()->first;
    return PLC_OK;
}

plc_status plc_trie_evict(plc_trie* t, int32_t id) {
    if (!t) return PLC_E_INVALID;
    auto it = t->end_of.find(id);
    if (it == t->end_of.end()) return PLC_E_INVALID;
    int cur = it->second;
    t->nodes[cur].terminals.erase(id);
    t->end_of.erase(it);
    while (cur != 0) {                       // drop the nodes no other stored prefix passes through
        const int parent = t->nodes[cur].parent;
        if (--t->nodes[cur].refs == 0) {
            t->nodes[parent].children.erase(t->nodes[cur].token);
            t->free_list.push_back(cur);
            t->live--;
        }
        cur = parent;
    }
    t->nodes[0].refs--;
    return PLC_OK;
}

plc_status plc_trie_stats(const plc_trie* t, int64_t* n_nodes, int64_t* n_prefixes) {
    if (!t || !n_nodes || !n_prefixes) return PLC_E_INVALID;
    *n_nodes = t->live;
    *n_prefixes = (int64_t)t->end_of.size();
    return PLC_OK;
}

}  // extern "C"
