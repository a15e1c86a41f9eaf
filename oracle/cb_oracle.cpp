// CPU oracle for the Cacheback draft-and-verify step.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, single-threaded statement of what the four library calls compute, written from the
// paper's description and sharing no code with the CUDA path.  Only tests, the smoke check and the
// benchmark's cpu-baseline leg may call it; the product path never does.
//
//   Table ........ Section 3.1 (cache table structure: leaders, followers, two LRU domains)
//   Update ....... Section 3.2 last paragraph + Section 3.3 last paragraph (sliding window over accepted
//                  tokens / over the prompt)
//   Draft tree ... Section 3.2 (recursive queries, breadth-first growth, TDL and CRT)
//   Frozen table . Section 3.3 (a read-only second table, queried after the dynamic one while the size cap allows)
//   Tree mask .... Section 3.2 (a token attends only to its ancestors)
//   Attention .... the textbook softmax(q.k * scale) v over the visible keys, in double precision
//   Acceptance ... Section 3.2 (one more token than the accepted draft tokens; longest verified branch)
//
// Readings taken where the paper is silent are marked "reading:" below.
// Parity pins: every function here is pinned by tests that do not go through this file's own formulas
// (hand traces, an OrderedDict model, brute force, torch CPU attention, closed forms). Nothing is unpinned.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <map>
#include <vector>

namespace {

using Key = std::vector<int32_t>;

struct Follower {
    Key tokens;          // FL tokens
    uint64_t stamp;      // recency inside this leader's follower list
};

struct Entry {
    uint64_t stamp;                  // leader recency
    std::vector<Follower> followers; // at most FC, unordered; order is defined by the stamps
};

struct Table {
    int LL, FL, LC, FC;
    bool refresh_on_reinsert;        // reading: re-observing a stored follower refreshes its recency
    uint64_t clock = 0;              // incremented by every insert and every query
    std::map<Key, Entry> leaders;

    // Section 3.1, insertion rule: a (leader, follower) pair creates the leader with that follower, or appends / refreshes the follower.
    void insert(const int32_t* L, const int32_t* F) {
        clock++;
        Key lk(L, L + LL), fk(F, F + FL);
        auto it = leaders.find(lk);
        if (it != leaders.end()) {
            Entry& e = it->second;
            e.stamp = clock;                                  // inserting a leader updates its recency
            for (auto& f : e.followers) {
                if (f.tokens == fk) {                         // already present: nothing is appended
                    if (refresh_on_reinsert) f.stamp = clock;
                    return;
                }
            }
            if ((int)e.followers.size() == FC) {              // evict the leader's LRU follower
                size_t v = 0;
                for (size_t i = 1; i < e.followers.size(); i++)
                    if (e.followers[i].stamp < e.followers[v].stamp) v = i;
                e.followers.erase(e.followers.begin() + v);
            }
            e.followers.push_back({fk, clock});
        } else {
            if ((int)leaders.size() == LC) {                  // evict the LRU leader with its followers
                auto v = leaders.begin();
                for (auto j = leaders.begin(); j != leaders.end(); ++j)
                    if (j->second.stamp < v->second.stamp) v = j;
                leaders.erase(v);
            }
            Entry e;
            e.stamp = clock;
            e.followers.push_back({fk, clock});
            leaders.emplace(std::move(lk), std::move(e));
        }
    }

    // Section 3.1: a query returns the followers (or nothing) and updates the leader's recency only.
    // reading: the list is returned most recently inserted first.
    std::vector<Key> query(const int32_t* L) {
        clock++;
        Key lk(L, L + LL);
        auto it = leaders.find(lk);
        if (it == leaders.end()) return {};
        it->second.stamp = clock;
        std::vector<const Follower*> fs;
        for (auto& f : it->second.followers) fs.push_back(&f);
        std::sort(fs.begin(), fs.end(), [](const Follower* a, const Follower* b) { return a->stamp > b->stamp; });
        std::vector<Key> out;
        for (auto* f : fs) out.push_back(f->tokens);
        return out;
    }
};

// Section 3.3: the frozen table is filled offline and never changes during decoding; a query returns the
// stored follower list as it is (reading: most frequent first, the order the builder stored) and has no side effect.
struct Frozen {
    int LL, FL;
    std::map<Key, std::vector<Key>> leaders;
};

inline double bf16_to_double(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return (double)f;
}

}  // namespace

extern "C" {

void* orc_table_new(int LL, int FL, int LC, int FC, int refresh_on_reinsert) {
    Table* t = new Table();
    t->LL = LL; t->FL = FL; t->LC = LC; t->FC = FC;
    t->refresh_on_reinsert = refresh_on_reinsert != 0;
    return t;
}
void orc_table_free(void* h) { delete (Table*)h; }
void orc_table_reset(void* h) { Table* t = (Table*)h; t->leaders.clear(); t->clock = 0; }
uint64_t orc_table_clock(void* h) { return ((Table*)h)->clock; }
int64_t orc_table_num_leaders(void* h) { return (int64_t)((Table*)h)->leaders.size(); }

void orc_insert(void* h, const int32_t* L, const int32_t* F) { ((Table*)h)->insert(L, F); }

// out: FC*FL tokens, followers most recent first. Returns the number of followers.
int orc_query(void* h, const int32_t* L, int32_t* out) {
    Table* t = (Table*)h;
    auto fs = t->query(L);
    for (size_t i = 0; i < fs.size(); i++) std::copy(fs[i].begin(), fs[i].end(), out + i * t->FL);
    return (int)fs.size();
}

// Sliding window over the tokens s[0..n_new): every leader-follower pair whose last token is new, i.e.
// whose window [i, i+LL+FL) ends in [n_old, n_new), is inserted in increasing i.
// reading: only complete windows of LL+FL tokens are inserted. Prompt initialisation is n_old = 0.
void orc_update(void* h, const int32_t* s, int n_old, int n_new) {
    Table* t = (Table*)h;
    const int w = t->LL + t->FL;
    int first = std::max(0, n_old - w + 1);
    for (int i = first; i + w <= n_new; i++) t->insert(s + i, s + i + t->LL);
}

// Canonical dump: leaders by increasing recency; each leader's followers by increasing recency.
// leaders: n*LL, nfol: n, followers: n*FC*FL (unused tail -1). Any pointer may be NULL. Returns n.
int64_t orc_table_dump(void* h, int32_t* leaders, int32_t* nfol, int32_t* followers) {
    Table* t = (Table*)h;
    std::vector<std::pair<uint64_t, const Key*>> order;
    for (auto& kv : t->leaders) order.push_back({kv.second.stamp, &kv.first});
    std::sort(order.begin(), order.end());
    int64_t n = 0;
    for (auto& o : order) {
        const Entry& e = t->leaders.at(*o.second);
        if (leaders) std::copy(o.second->begin(), o.second->end(), leaders + n * t->LL);
        if (nfol) nfol[n] = (int32_t)e.followers.size();
        if (followers) {
            std::vector<const Follower*> fs;
            for (auto& f : e.followers) fs.push_back(&f);
            std::sort(fs.begin(), fs.end(), [](const Follower* a, const Follower* b) { return a->stamp < b->stamp; });
            int32_t* dst = followers + n * t->FC * t->FL;
            std::fill(dst, dst + t->FC * t->FL, -1);
            for (size_t i = 0; i < fs.size(); i++) std::copy(fs[i]->tokens.begin(), fs[i]->tokens.end(), dst + i * t->FL);
        }
        n++;
    }
    return n;
}

// Draft-tree growth (Section 3.2).  Node 0 is the last token of the sequence (the one token that is not
// KV-cached yet; reading: exactly one such token, counted in the size cap T).  Level 1 queries the last
// LL tokens of the sequence; each later level queries, for every leaf that ended a complete follower,
// the last LL tokens of (sequence ++ path to the leaf).  Growth is breadth first, leaves in order, each
// leaf's followers most recent first; it stops at T nodes or when no leaf has a follower.
// readings: level 1 may use at most T - crt nodes (crt tokens stay reserved for deeper levels); a
// follower that does not fit the remaining room or the depth cap is cut short and never grown further;
// no query is issued once the level's cap is reached; a key that would need tokens before the start of
// the sequence is not queried.
// Outputs are padded with -1 (mask rows with 0) beyond n.  query_log (optional) receives, per issued
// query, LL key tokens followed by the hit count.  Returns n.
// Dual-table form (Section 3.3): when a frozen table is given, the dynamic table forms the tree first, as above;
// then, if the tree is still below T nodes, growth continues from the frozen table.
// readings: the frozen pass visits, first in first out, every node at which a follower list can be attached (the
// root and the last node of every complete follower, in the order they were created), and the ends of the
// complete followers it adds itself join the queue; a query at the root is issued, and its followers appended,
// only while the tree has fewer than max(1, T - crt) nodes, any other only while it has fewer than T (the same
// rule that the dynamic pass follows, whose level 1 is the root alone); frozen followers are appended most
// frequent first and are not compared with the branches already present; frozen queries neither tick the
// dynamic table's clock nor touch any recency.  frozen_log (optional): per issued frozen query, LL key tokens
// followed by the hit count.
static int draft_impl(Table* t, const Frozen* fz, const int32_t* s, int seq_len, int T, int crt, int max_depth,
                      int32_t* tok, int32_t* par, int32_t* dep, uint32_t* mask, int32_t* query_log,
                      int32_t* n_queries, int32_t* frozen_log, int32_t* n_frozen_queries) {
    const int LL = t->LL, FL = t->FL, W = (T + 31) / 32;
    std::fill(tok, tok + T, -1);
    std::fill(par, par + T, -1);
    std::fill(dep, dep + T, -1);
    std::fill(mask, mask + (size_t)T * W, 0u);
    int nq = 0, nfq = 0;
    if (n_queries) *n_queries = 0;
    if (n_frozen_queries) *n_frozen_queries = 0;
    if (seq_len < 1 || T < 1) return 0;
    int n = 1;
    tok[0] = s[seq_len - 1]; par[0] = -1; dep[0] = 0;
    // key = last LL tokens of sequence[0..seq_len-1) ++ tokens on root->leaf (root = s[seq_len-1])
    auto make_key = [&](int leaf, Key& key) {
        bool ok = true;
        std::vector<int32_t> path;                               // leaf up to root
        for (int c = leaf; c >= 0; c = par[c]) path.push_back(tok[c]);
        for (int j = 0; j < LL; j++) {                            // j-th token from the end
            int32_t v;
            if (j < (int)path.size()) v = path[j];
            else {
                int pos = seq_len - 1 - (j - ((int)path.size() - 1));
                v = pos >= 0 ? s[pos] : -1;
            }
            if (v < 0) ok = false;
            key[LL - 1 - j] = v;
        }
        return ok;
    };
    // appends the followers fs below leaf while fewer than cap nodes exist; complete ones are reported through ends
    auto attach = [&](int leaf, const std::vector<Key>& fs, int cap, std::vector<int>& ends) {
        for (auto& F : fs) {
            if (n >= cap) break;
            int p = leaf, k = 0;
            for (int j = 0; j < FL; j++) {
                if (n >= cap || dep[p] >= max_depth) break;
                tok[n] = F[j]; par[n] = p; dep[n] = dep[p] + 1; p = n; n++; k++;
            }
            if (k == FL) ends.push_back(p);
        }
    };
    std::vector<int> points{0};                                  // every node that ever was a frontier leaf
    std::vector<int> frontier{0};
    int level = 1;
    while (!frontier.empty() && n < T) {
        const int cap = (level == 1) ? std::max(1, T - crt) : T;
        std::vector<int> next;
        for (int leaf : frontier) {
            if (n >= cap) break;
            if (dep[leaf] >= max_depth) continue;
            Key key(LL);
            if (!make_key(leaf, key)) continue;
            auto fs = t->query(key.data());
            if (query_log) {
                std::copy(key.begin(), key.end(), query_log + (size_t)nq * (LL + 1));
                query_log[(size_t)nq * (LL + 1) + LL] = (int32_t)fs.size();
            }
            nq++;
            attach(leaf, fs, cap, next);
        }
        points.insert(points.end(), next.begin(), next.end());
        frontier.swap(next);
        level++;
    }
    if (fz) {
        for (size_t qi = 0; qi < points.size() && n < T; qi++) {  // the queue grows while it is walked
            const int leaf = points[qi];
            const int cap = leaf == 0 ? std::max(1, T - crt) : T;
            if (n >= cap) continue;
            if (dep[leaf] >= max_depth) continue;
            Key key(LL);
            if (!make_key(leaf, key)) continue;
            auto it = fz->leaders.find(key);
            const std::vector<Key> none;
            const std::vector<Key>& fs = it == fz->leaders.end() ? none : it->second;
            if (frozen_log) {
                std::copy(key.begin(), key.end(), frozen_log + (size_t)nfq * (LL + 1));
                frozen_log[(size_t)nfq * (LL + 1) + LL] = (int32_t)fs.size();
            }
            nfq++;
            std::vector<int> ends;
            attach(leaf, fs, cap, ends);
            points.insert(points.end(), ends.begin(), ends.end());
        }
    }
    // Tree mask: a token attends to itself and its ancestors, root included.
    for (int i = 0; i < n; i++) {
        if (par[i] >= 0) std::copy(mask + (size_t)par[i] * W, mask + (size_t)par[i] * W + W, mask + (size_t)i * W);
        mask[(size_t)i * W + i / 32] |= 1u << (i % 32);
    }
    if (n_queries) *n_queries = nq;
    if (n_frozen_queries) *n_frozen_queries = nfq;
    return n;
}

int orc_draft_tree(void* h, const int32_t* s, int seq_len, int T, int crt, int max_depth,
                   int32_t* tok, int32_t* par, int32_t* dep, uint32_t* mask, int32_t* query_log,
                   int32_t* n_queries) {
    return draft_impl((Table*)h, nullptr, s, seq_len, T, crt, max_depth, tok, par, dep, mask, query_log, n_queries, nullptr, nullptr);
}

void* orc_frozen_new(int LL, int FL) {
    Frozen* f = new Frozen();
    f->LL = LL; f->FL = FL;
    return f;
}
void orc_frozen_free(void* h) { delete (Frozen*)h; }
// One leader with its nf followers (nf * FL tokens), most frequent first.
void orc_frozen_add(void* h, const int32_t* L, int nf, const int32_t* followers) {
    Frozen* f = (Frozen*)h;
    std::vector<Key> fs;
    for (int i = 0; i < nf; i++) fs.emplace_back(followers + (size_t)i * f->FL, followers + (size_t)(i + 1) * f->FL);
    f->leaders[Key(L, L + f->LL)] = std::move(fs);
}
int orc_draft_tree_dual(void* h, void* hf, const int32_t* s, int seq_len, int T, int crt, int max_depth,
                        int32_t* tok, int32_t* par, int32_t* dep, uint32_t* mask, int32_t* query_log,
                        int32_t* n_queries, int32_t* frozen_log, int32_t* n_frozen_queries) {
    return draft_impl((Table*)h, (const Frozen*)hf, s, seq_len, T, crt, max_depth, tok, par, dep, mask, query_log, n_queries,
                      frozen_log, n_frozen_queries);
}

// Ancestor-or-self mask of a given tree (parents precede children).
void orc_tree_mask(const int32_t* par, int n, int T, uint32_t* mask) {
    const int W = (T + 31) / 32;
    std::fill(mask, mask + (size_t)T * W, 0u);
    for (int i = 0; i < n; i++) {
        if (par[i] >= 0) std::copy(mask + (size_t)par[i] * W, mask + (size_t)par[i] * W + W, mask + (size_t)i * W);
        mask[(size_t)i * W + i / 32] |= 1u << (i % 32);
    }
}

// Greedy target of each row: index of the first (lowest-index) maximum. reading: ties go to the lowest id.
void orc_argmax_f32(const float* logits, int rows, int64_t row_stride, int V, int32_t* out) {
    for (int r = 0; r < rows; r++) {
        const float* x = logits + (int64_t)r * row_stride;
        int best = 0;
        for (int v = 1; v < V; v++) if (x[v] > x[best]) best = v;
        out[r] = best;
    }
}

// Greedy acceptance (Section 3.2): a node is verified when its parent is verified and its token equals
// the target's choice after the parent; the deepest verified node wins (reading: smallest index among
// equally deep ones); the step emits the tokens on the path below the root plus the target's choice after
// the last accepted node, i.e. between 1 and 1 + longest-branch tokens.
// accept_nodes: dmax entries, out_tokens: dmax+1 entries, both padded with -1. Returns the number of
// accepted draft tokens m (the step emits m + 1 tokens).
int orc_accept(const int32_t* tok, const int32_t* par, const int32_t* dep, int n, const int32_t* target,
               int dmax, int32_t* accept_nodes, int32_t* out_tokens) {
    std::fill(accept_nodes, accept_nodes + dmax, -1);
    std::fill(out_tokens, out_tokens + dmax + 1, -1);
    if (n < 1) return 0;
    std::vector<char> ok(n, 0);
    ok[0] = 1;
    int best = 0;
    for (int i = 1; i < n; i++) {
        ok[i] = ok[par[i]] && tok[i] == target[par[i]];
        if (ok[i] && dep[i] > dep[best]) best = i;
    }
    int m = dep[best];
    for (int c = best, k = m - 1; c > 0; c = par[c], k--) { accept_nodes[k] = c; out_tokens[k] = tok[c]; }
    out_tokens[m] = target[best];
    return m;
}

// Tree-masked attention, plain definition in double precision, for selected output rows.
//   q        bf16 bits [B, T, Hq, D]
//   k_pool, v_pool bf16 bits [num_pages, P, Hkv, D]; block_table int32 [B, max_pages]; ctx_len int32 [B]
//   k_tree, v_tree bf16 bits [B, T, Hkv, D]; tree_mask uint32 [B, T, W]
//   rows     int32 [n_rows, 3] = (b, q_head, node)
//   out      double [n_rows, D]; lse double [n_rows] (natural log)
// Node i of sequence b sees every cached key t < ctx_len[b] of kv head h / (Hq/Hkv), plus the tree keys j
// whose bit is set in its mask row.  reading: scale is given by the caller (1/sqrt(D) by default).
void orc_tree_attn_rows(const uint16_t* q, const uint16_t* k_pool, const uint16_t* v_pool,
                        const int32_t* block_table, const int32_t* ctx_len, const uint16_t* k_tree,
                        const uint16_t* v_tree, const uint32_t* tree_mask, int T, int Hq, int Hkv, int D,
                        int P, int max_pages, double scale, const int32_t* rows, int n_rows, double* out,
                        double* lse) {
    const int G = Hq / Hkv, W = (T + 31) / 32;
    for (int r = 0; r < n_rows; r++) {
        const int b = rows[3 * r], h = rows[3 * r + 1], i = rows[3 * r + 2], kh = h / G;
        const uint16_t* qv = q + (((size_t)b * T + i) * Hq + h) * D;
        std::vector<double> s;
        std::vector<const uint16_t*> vrow;
        for (int t = 0; t < ctx_len[b]; t++) {
            size_t page = (size_t)block_table[(size_t)b * max_pages + t / P];
            size_t off = ((page * P + t % P) * Hkv + kh) * D;
            double acc = 0;
            for (int d = 0; d < D; d++) acc += bf16_to_double(qv[d]) * bf16_to_double(k_pool[off + d]);
            s.push_back(acc * scale);
            vrow.push_back(v_pool + off);
        }
        for (int j = 0; j < T; j++) {
            if (!((tree_mask[((size_t)b * T + i) * W + j / 32] >> (j % 32)) & 1u)) continue;
            size_t off = (((size_t)b * T + j) * Hkv + kh) * D;
            double acc = 0;
            for (int d = 0; d < D; d++) acc += bf16_to_double(qv[d]) * bf16_to_double(k_tree[off + d]);
            s.push_back(acc * scale);
            vrow.push_back(v_tree + off);
        }
        double m = -std::numeric_limits<double>::infinity();
        for (double x : s) m = std::max(m, x);
        double sum = 0;
        for (double x : s) sum += std::exp(x - m);
        for (int d = 0; d < D; d++) out[(size_t)r * D + d] = 0;
        for (size_t j = 0; j < s.size(); j++) {
            double p = std::exp(s[j] - m) / sum;
            for (int d = 0; d < D; d++) out[(size_t)r * D + d] += p * bf16_to_double(vrow[j][d]);
        }
        if (lse) lse[r] = m + std::log(sum);
    }
}

}  // extern "C"
