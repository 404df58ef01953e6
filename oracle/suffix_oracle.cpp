// CPU oracle for SuffixDecoding draft generation.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, pointer-based implementation of what the paper's Section 3
// and Algorithm 1 compute, written to be checked against the paper by eye.
// It shares no code with the CUDA library and must never be called from the
// product path: only tests, the smoke check and the benchmark's CPU-baseline
// leg may load it.
//
// Readings of the paper taken here (each is also listed in the design notes):
//  * Store (Section 3, "Suffix Tree Construction"; COUNT below Eq. 2): one
//    node per token; the path root->node is a token string of length <= D and
//    COUNT(node) is the number of occurrences of that string in the corpus.
//    Strings never cross a sequence boundary.  D (depth cap) is an added limit.
//  * MatchPattern (Algorithm 1): walk the last p tokens from the root.
//  * C(N), D(N) (Eq. 1, Eq. 2): C = COUNT(N) / sum of COUNT over N's siblings
//    including N; D = D(parent) * C, D(N_p) = 1.
//  * ExpandSpeculationTree (Algorithm 1): best-first growth.  The candidate
//    set is every not-yet-added child of any node already in the tree; the
//    budget counts draft nodes only (N_p is the known last token).
//  * SCORE (Eq. 4) sums D over draft nodes in the order they were added.
//  * MAX_SPEC(p) = floor(alpha * p) (Eq. 3), additionally capped.
//  * GenerateCandidateTree (Algorithm 1): global tree first, then the
//    per-request tree, p ascending, strict '>' from 0.
//  * Ties between candidates: higher D, then lower token id, then lower index
//    of the parent inside the speculation tree (N_p counts as -1).
//  * fp64 throughout; divide, then multiply root-to-leaf; no fused multiply-add
//    (compile with -ffp-contract=off).
//
// Parity pins (tests/test_oracle_*.py): counts against brute-force substring
// counting, closed forms for a^L / all-distinct / k-fold corpora, expansion
// against exhaustive search over connected sub-trees, hand-built tie cases,
// mask/position invariants, the prompt-lookup special case.  Which tree wins
// on realistic data has no independent pin ("parity unpinned" beyond those).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <map>
#include <queue>
#include <thread>
#include <vector>

namespace {

struct Node {
    int32_t count = 0;
    std::map<int32_t, Node*> children;   // ordered by token id
};

void destroy(Node* n) {
    for (auto& kv : n->children) { destroy(kv.second); delete kv.second; }
    n->children.clear();
}

// Add one occurrence of the string s[0..len) (len <= D): COUNT of every node on
// the path grows by one.  Used once per suffix start by a whole-sequence insert.
void add_path(Node* root, const int32_t* s, int64_t len) {
    Node* cur = root;
    for (int64_t k = 0; k < len; ++k) {
        Node*& slot = cur->children[s[k]];
        if (!slot) slot = new Node();
        cur = slot;
        cur->count += 1;
    }
}

// Add one occurrence of the string s[0..len): only its LAST node gains a count
// (the shorter prefixes were counted when their own last token arrived).
void add_last(Node* root, const int32_t* s, int64_t len) {
    Node* cur = root;
    for (int64_t k = 0; k < len; ++k) {
        Node*& slot = cur->children[s[k]];
        if (!slot) slot = new Node();
        cur = slot;
    }
    cur->count += 1;
}

struct Trie {
    Node root;
    int D = 32;
    ~Trie() { destroy(&root); }
    void clear() { destroy(&root); root.count = 0; }

    // Whole finished sequence: every start i contributes s[i .. min(i+D, n)).
    void insert_sequence(const int32_t* s, int64_t n) {
        for (int64_t i = 0; i < n; ++i) add_path(&root, s + i, std::min<int64_t>(D, n - i));
    }
    // Text grew to length t (token text[t-1] is new): every substring that ENDS at
    // the new token and has length <= D occurs once more.
    void extend(const int32_t* text, int64_t t) {
        for (int64_t len = 1; len <= std::min<int64_t>(D, t); ++len) add_last(&root, text + (t - len), len);
    }
    const Node* walk(const int32_t* s, int64_t len) const {
        const Node* cur = &root;
        for (int64_t k = 0; k < len; ++k) {
            auto it = cur->children.find(s[k]);
            if (it == cur->children.end()) return nullptr;
            cur = it->second;
        }
        return cur;
    }
};

struct Draft {               // one node of a speculation tree, in insertion order
    int32_t token;
    int32_t parent;          // index in the tree; -1: child of N_p
    double d;                // D(N), Eq. 2
};

struct Candidate {
    double d;
    int32_t token;
    int32_t parent;
    const Node* node;
};
struct Worse {               // a is worse than b  (priority_queue keeps the best on top)
    bool operator()(const Candidate& a, const Candidate& b) const {
        if (a.d != b.d) return a.d < b.d;
        if (a.token != b.token) return a.token > b.token;
        return a.parent > b.parent;
    }
};

void push_children(std::priority_queue<Candidate, std::vector<Candidate>, Worse>& pq, const Node* q,
                   double d_parent, int32_t parent_index) {
    int64_t sum = 0;                                   // denominator of Eq. 1
    for (auto& kv : q->children) sum += kv.second->count;
    for (auto& kv : q->children) {
        double c = (double)kv.second->count / (double)sum;      // Eq. 1
        double d = d_parent * c;                                // Eq. 2
        pq.push(Candidate{d, kv.first, parent_index, kv.second});
    }
}

// ExpandSpeculationTree(N_p, budget); returns SCORE (Eq. 4).  linear=true keeps only
// the chain variant: every new node must be a child of the previously added one.
double expand(const Node* np, int budget, bool linear, std::vector<Draft>& out) {
    out.clear();
    double score = 0.0;
    if (!np || budget <= 0) return score;
    std::priority_queue<Candidate, std::vector<Candidate>, Worse> pq;
    push_children(pq, np, 1.0, -1);
    while ((int)out.size() < budget && !pq.empty()) {
        Candidate c = pq.top();
        pq.pop();
        int32_t idx = (int32_t)out.size();
        out.push_back(Draft{c.token, c.parent, c.d});
        score = score + c.d;
        if (linear) pq = std::priority_queue<Candidate, std::vector<Candidate>, Worse>();
        push_children(pq, c.node, c.d, idx);
    }
    return score;
}

int budget_for(double alpha, int p, int cap) {
    double b = std::floor(alpha * (double)p);          // Eq. 3
    if (b > (double)cap) return cap;
    if (b < 0.0) return 0;
    return (int)b;
}

struct Slot {
    Trie trie;
    std::vector<int32_t> text;
    int64_t updates = 0;     // nodes whose COUNT grew through appends (one per string that ends at a new token)
};

struct Oracle {
    int D;
    Trie global;
    std::vector<Slot> slots;
};

enum { FLAG_GLOBAL_ONLY = 1, FLAG_REQUEST_ONLY = 2, FLAG_LINEAR = 4 };

struct SpecOut {
    int32_t* n_draft; int32_t* tokens; int32_t* parents; int32_t* positions; uint32_t* mask;
    int32_t* chosen_tree; int32_t* chosen_p; double* score; int64_t* visited;
};

// The node of pattern `pat` (p tokens) in S, or null.  `steps` grows by one for every child that
// was found on the way (the work counter "descents": a pattern that fails at its k-th token adds k - 1).
const Node* match_counting(const Trie& S, const int32_t* pat, int p, int64_t& steps) {
    const Node* n = &S.root;
    for (int k = 0; k < p; ++k) {
        auto it = n->children.find(pat[k]);
        if (it == n->children.end()) return nullptr;
        n = it->second;
        ++steps;
    }
    return n;
}

struct TreeCandidate {       // one speculation tree that Section 3's selection step looks at
    int tree, p;             // where it came from: 0 global / 1 per-request, pattern length
    double score;            // Eq. 4
    std::vector<Draft> drafts;
};

// Candidate selection for one request (Section 3, "Speculation Tree Scoring" and the adaptive
// budget of Eq. 3), then the arrays the verifier takes.  Two stages: every (tree, pattern length)
// pair that matches yields one scored tree; then the first tree with the strictly largest score
// is kept, provided it beats the threshold of Section 3.2.
void speculate_one(const Oracle& o, int i, int slot, int P, double alpha, int cap, int flags, int M,
                   const int32_t* budget_override, double tau, const SpecOut& r) {
    const Slot& s = o.slots[slot];
    const int64_t t = (int64_t)s.text.size();
    const int words = (M + 31) / 32;
    int cap_i = cap;
    if (budget_override && budget_override[i] >= 0) cap_i = std::min(cap, (int)budget_override[i]);
    const bool linear = (flags & FLAG_LINEAR) != 0;

    // stage 1: the candidates, global tree before per-request tree, short patterns before long ones
    std::vector<TreeCandidate> cands;
    int64_t descents = 0, adds = 0;
    for (int tree = 0; tree < 2; ++tree) {
        if (tree == 0 && (flags & FLAG_REQUEST_ONLY)) continue;
        if (tree == 1 && (flags & FLAG_GLOBAL_ONLY)) continue;
        const Trie& S = tree == 0 ? o.global : s.trie;
        const int p_max = (int)std::min<int64_t>(std::min<int64_t>(P, t), o.D);
        for (int p = 1; p <= p_max; ++p) {
            const Node* np = match_counting(S, s.text.data() + (t - p), p, descents);
            if (!np) continue;
            TreeCandidate c{tree, p, 0.0, {}};
            c.score = expand(np, budget_for(alpha, p, cap_i), linear, c.drafts);
            adds += (int64_t)c.drafts.size();
            cands.push_back(std::move(c));
        }
    }
    // stage 2: the best one; equal scores keep the earlier candidate, a score of 0 is no candidate
    const TreeCandidate* best = nullptr;
    double best_score = 0.0;
    for (const TreeCandidate& c : cands)
        if (c.score > best_score) { best_score = c.score; best = &c; }
    // Section 3.2 ("Hybrid Suffix Speculative Decoding"): the suffix tree's draft is used only if
    // its score exceeds the threshold tau; otherwise the caller falls back to its other drafter.
    if (best && !(best_score > tau)) { best = nullptr; best_score = 0.0; }

    const int n = best ? (int)best->drafts.size() : 0;
    r.n_draft[i] = n; r.chosen_tree[i] = best ? best->tree : -1; r.chosen_p[i] = best ? best->p : 0;
    r.score[i] = best_score;
    if (r.visited) {
        // measurement only: descents of all matches, nodes added to all candidate trees, and the
        // number of candidate trees (matched (tree, p) pairs that got at least one draft node)
        int64_t trees = 0;
        for (const TreeCandidate& c : cands) trees += c.drafts.empty() ? 0 : 1;
        r.visited[3 * i] = descents; r.visited[3 * i + 1] = adds; r.visited[3 * i + 2] = trees;
    }
    int32_t* tok = r.tokens + (int64_t)i * M; int32_t* par = r.parents + (int64_t)i * M;
    int32_t* pos = r.positions + (int64_t)i * M; uint32_t* msk = r.mask + (int64_t)i * M * words;
    std::vector<int> depth(M, 0);
    for (int j = 0; j < M; ++j) { tok[j] = -1; par[j] = -1; pos[j] = -1; }
    std::memset(msk, 0, sizeof(uint32_t) * (size_t)M * words);
    for (int j = 0; j < n; ++j) {
        tok[j] = best->drafts[j].token; par[j] = best->drafts[j].parent;
        depth[j] = par[j] < 0 ? 1 : depth[par[j]] + 1;
        pos[j] = (int32_t)(t + depth[j] - 1);
        for (int a = j; a >= 0; a = par[a]) msk[(int64_t)j * words + a / 32] |= (1u << (a % 32));
    }
}

}  // namespace

extern "C" {

void* sfx_oracle_create(int depth_cap, int n_slots) {
    Oracle* o = new Oracle();
    o->D = depth_cap; o->global.D = depth_cap;
    o->slots = std::vector<Slot>(n_slots);
    for (auto& s : o->slots) s.trie.D = depth_cap;
    return o;
}
void sfx_oracle_destroy(void* h) { delete (Oracle*)h; }

void sfx_oracle_global_insert(void* h, const int32_t* tok, int64_t n) { ((Oracle*)h)->global.insert_sequence(tok, n); }

void sfx_oracle_slot_reset(void* h, int slot) {
    Slot& s = ((Oracle*)h)->slots[slot];
    s.trie.clear(); s.text.clear(); s.updates = 0;
}
void sfx_oracle_slot_append(void* h, int slot, const int32_t* tok, int64_t n) {
    Slot& s = ((Oracle*)h)->slots[slot];
    for (int64_t k = 0; k < n; ++k) {
        s.text.push_back(tok[k]);
        s.trie.extend(s.text.data(), (int64_t)s.text.size());
        s.updates += std::min<int64_t>(s.trie.D, (int64_t)s.text.size());
    }
}
// Several slots at once, one thread per group of slots (slots are independent).
void sfx_oracle_slot_append_batch(void* h, int n, const int32_t* slots, const int64_t* offsets,
                                  const int32_t* tok, int n_threads) {
    if (n_threads < 1) n_threads = 1;
    std::vector<std::thread> th;
    for (int w = 0; w < n_threads; ++w)
        th.emplace_back([=] {
            for (int i = w; i < n; i += n_threads)
                sfx_oracle_slot_append(h, slots[i], tok + offsets[i], offsets[i + 1] - offsets[i]);
        });
    for (auto& x : th) x.join();
}
// Node updates the appends to this slot have made since its last reset: every appended token
// raises the COUNT of one node per string that ends at it (at most D of them).
int64_t sfx_oracle_slot_updates(void* h, int slot) { return ((Oracle*)h)->slots[slot].updates; }
int64_t sfx_oracle_slot_len(void* h, int slot) { return (int64_t)((Oracle*)h)->slots[slot].text.size(); }
void sfx_oracle_slot_text(void* h, int slot, int32_t* out) {
    Slot& s = ((Oracle*)h)->slots[slot];
    std::memcpy(out, s.text.data(), s.text.size() * sizeof(int32_t));
}

static const Trie& pick(Oracle* o, int tree) { return tree < 0 ? o->global : o->slots[tree].trie; }

// COUNT of the node reached by `path` in tree (-1: global, else slot); 0 if absent.
int64_t sfx_oracle_count(void* h, int tree, const int32_t* path, int len) {
    const Node* n = pick((Oracle*)h, tree).walk(path, len);
    return n ? n->count : 0;
}

static int64_t count_nodes(const Node* n) {
    int64_t c = 0;
    for (auto& kv : n->children) c += 1 + count_nodes(kv.second);
    return c;
}
int64_t sfx_oracle_node_count(void* h, int tree) { return count_nodes(&pick((Oracle*)h, tree).root); }

struct DumpCtx { int64_t cap, n; int32_t *depth, *parent, *tok, *cnt; };
static void dump_rec(const Node* n, int d, int32_t self, DumpCtx& c) {
    for (auto& kv : n->children) {
        int64_t id = c.n++;
        if (id < c.cap) { c.depth[id] = d + 1; c.parent[id] = self; c.tok[id] = kv.first; c.cnt[id] = kv.second->count; }
        dump_rec(kv.second, d + 1, (int32_t)id, c);
    }
}
// Pre-order listing (children by ascending token).  Returns the node count.
int64_t sfx_oracle_dump(void* h, int tree, int64_t cap, int32_t* depth, int32_t* parent, int32_t* tok, int32_t* cnt) {
    DumpCtx c{cap, 0, depth, parent, tok, cnt};
    dump_rec(&pick((Oracle*)h, tree).root, 0, -1, c);
    return c.n;
}

// One (tree, p) candidate for an explicit context x_{1:t}: MatchPattern then
// ExpandSpeculationTree.  Returns the number of draft nodes, -1 if no match.
int sfx_oracle_candidate(void* h, int tree, const int32_t* ctx, int64_t t, int p, int budget, int linear,
                         int32_t* tokens, int32_t* parents, double* dvals, double* score) {
    Oracle* o = (Oracle*)h;
    *score = 0.0;
    if (p > t || p > o->D || p < 1) return -1;
    const Node* n = pick(o, tree).walk(ctx + (t - p), p);
    if (!n) return -1;
    std::vector<Draft> out;
    *score = expand(n, budget, linear != 0, out);
    for (size_t j = 0; j < out.size(); ++j) { tokens[j] = out[j].token; parents[j] = out[j].parent; dvals[j] = out[j].d; }
    return (int)out.size();
}

// Empirical entropy (Appendix "Predicting SuffixDecoding Effectiveness"): entropy in bits of
// each node's children distribution, averaged with the children's total count as weight.
static void entropy_rec(const Node* n, double& acc, double& weight) {
    if (n->children.empty()) return;
    double sum = 0.0;
    for (auto& kv : n->children) sum += (double)kv.second->count;
    double h = 0.0;
    for (auto& kv : n->children) {
        double p = (double)kv.second->count / sum;
        h -= p * std::log2(p);
    }
    acc += sum * h;
    weight += sum;
    for (auto& kv : n->children) entropy_rec(kv.second, acc, weight);
}
double sfx_oracle_entropy(void* h, int tree) {
    double acc = 0.0, weight = 0.0;
    entropy_rec(&pick((Oracle*)h, tree).root, acc, weight);
    return weight > 0.0 ? acc / weight : 0.0;
}

int sfx_oracle_budget(double alpha, int p, int cap) { return budget_for(alpha, p, cap); }

// GenerateCandidateTree for n requests.  Row stride of every per-draft output is M.
void sfx_oracle_speculate(void* h, int n, const int32_t* slots, int P, double alpha, int max_spec, int flags,
                          int M, const int32_t* budget_override, int32_t* n_draft, int32_t* tokens,
                          int32_t* parents, int32_t* positions, uint32_t* mask, int32_t* chosen_tree,
                          int32_t* chosen_p, double* score, int64_t* visited, int n_threads, double tau) {
    Oracle* o = (Oracle*)h;
    SpecOut r{n_draft, tokens, parents, positions, mask, chosen_tree, chosen_p, score, visited};
    if (n_threads <= 1) {
        for (int i = 0; i < n; ++i) speculate_one(*o, i, slots[i], P, alpha, max_spec, flags, M, budget_override, tau, r);
        return;
    }
    std::vector<std::thread> th;
    for (int w = 0; w < n_threads; ++w)
        th.emplace_back([=] {
            for (int i = w; i < n; i += n_threads)
                speculate_one(*o, i, slots[i], P, alpha, max_spec, flags, M, budget_override, tau, r);
        });
    for (auto& x : th) x.join();
}

}  // extern "C"
