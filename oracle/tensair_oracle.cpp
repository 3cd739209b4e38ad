// CPU oracle for the SGNS mini-batch step and the DASGD exchange of sparse gradient messages.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the CUDA library is
// checked against.  It shares no code with the CUDA path and must never be called from it; only
// the tests, the smoke check and the CPU-baseline leg of the benchmark load it.
//
// What it follows:
//   * Eq. 1 of the paper: theta_{t+1} = theta_t - alpha * grad L(X, theta_t).  The gradient of the
//     WHOLE mini-batch is evaluated at the single snapshot theta_t; nothing is updated mid-batch.
//   * Section 2.2 "gradient calculation" (GC) vs "gradient application" (GA): train_batch = GC +
//     local GA; apply_messages = GA of gradients received from other Model instances.
//   * Algorithm 1, procedure train: mini-batch branch (compute, apply locally, buffer, send when the
//     buffer holds maxGradBuffer gradients; here maxGradBuffer = 1) and gradient branch (apply a
//     received gradient as it stands).
//   * Section 3.1 (model consistency): processing order inside one Model and the staleness metric
//     |G_i u G_j| - |G_i n G_j|, G_i taken when the gradient is computed, G_j when it is applied.
//   * The loss is the textbook skip-gram negative-sampling objective (the paper only names "a
//     default skip-gram model"): per pair  -log s(u_o.v_c) - sum_j log s(-u_nj.v_c).
//
// With maxGradBuffer = m > 1 a replica sends only after every m-th mini-batch: the sum of the m buffered
// gradient messages over the union of their rows (fp32 additions in the order computed).  The
// staleness snapshot G_i of such a message is taken when it is sent.
//
// Routed mini-batches (Section 4.3: the (x, y) pairs are spread over the Model instances by a hash
// partitioner keyed by the word x): every replica is handed the same token batch and trains the pairs
// whose centre word is routed to it, route(x) = mulhi32(Philox(x, 0, 0, tag 4; seed).word0, W).  The
// replicas then compute disjoint parts of ONE mini-batch gradient: pair indices, negative draws
// (replica tag 0) and the mean's denominator are those of the whole batch, so the routed messages of
// the W replicas add up to the message a single model computes from that batch.
//
// Arithmetic: tables are stored in fp32; every dot product, sigmoid, loss term and gradient sum is
// taken in fp64 from those fp32 values; a delta row is fp32(-scale * sum) with scale = (double)lr when
// the batch loss is the sum of the pair losses and (double)lr / (number of pairs) when it is their
// mean (the paper does not say which; its footnoted Keras model averages over the batch); applying a
// delta is one fp32 addition per element.
//
// Pins (see tests/): Philox known-answer vectors; alias-table exact reconstruction, equal-count
// special case and chi-square; single-pair closed form; batch-0 closed form; central finite
// differences; brute-force pair enumeration and touched-row sets; the staleness values 0 / 2 / 3 of
// the paper's Fig. 2 example; W = 1 == plain SGD; exactly-once delivery; replica agreement after a
// drain.  Parity unpinned: long runs (hundreds of batches) and drift runs have no independent pin
// beyond loss sanity (starts at (1+k) ln 2 per pair, decreases).
//
// OpenMP is used only over independent items (pairs for the scalars, distinct rows for the sums), so
// results do not depend on the thread count.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <deque>
#include <map>
#include <set>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11)
// ---------------------------------------------------------------------------------------------
struct U4 { uint32_t v[4]; };

U4 philox4x32_10(U4 ctr, uint32_t k0, uint32_t k1) {
    for (int round = 0; round < 10; ++round) {
        uint64_t prod_a = (uint64_t)0xD2511F53u * ctr.v[0];
        uint64_t prod_b = (uint64_t)0xCD9E8D57u * ctr.v[2];
        U4 nxt;
        nxt.v[0] = (uint32_t)(prod_b >> 32) ^ ctr.v[1] ^ k0;
        nxt.v[1] = (uint32_t)prod_b;
        nxt.v[2] = (uint32_t)(prod_a >> 32) ^ ctr.v[3] ^ k1;
        nxt.v[3] = (uint32_t)prod_a;
        ctr = nxt;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return ctr;
}

enum : uint32_t { TAG_NEGATIVE = 1, TAG_DELAY = 2, TAG_INIT = 3, TAG_ROUTE = 4 };

inline uint32_t mulhi32(uint32_t a, uint32_t b) { return (uint32_t)(((uint64_t)a * b) >> 32); }

// ---------------------------------------------------------------------------------------------
// Walker alias table over weights count^0.75, built in exact integer arithmetic
// ---------------------------------------------------------------------------------------------
// The paper does not describe the negative sampler; the table is defined here so that its result does
// not depend on the order in which a builder visits the entries (a sequential sweep, as below, and a
// parallel builder working from prefix sums must produce the same bits).
//   weight_i = s*s*s, s = sqrt(sqrt(count_i))      (fp64; square roots are correctly rounded, pow is not)
//   u_i      = floor(weight_i * 2^sh), sh = bits - e, 2^(e-1) <= max weight < 2^e,
//              bits = min(42, 62 - ceil(log2 V))    (integer masses below 2^bits)
//   C        = ceil(sum u / V); the first entry of largest u takes C*V - sum u more, so that sum u = C*V:
//              V buckets of capacity C.
// Entries with u < C are light, the others heavy, each kind in ascending index order.  The current heavy
// entry h, with what is left of its mass r (at first u_h), tops up light buckets in order while r > C:
// light l keeps u_l of its bucket, alias[l] = h, r -= C - u_l.  Once r <= C the heavy entry's own bucket
// is closed with r of its own mass, topped up by the next heavy entry h' (alias[h] = h'), which goes on
// with r' = u_h' - (C - r).  A bucket keeping all of C accepts always (thresh all-ones, alias = itself);
// otherwise thresh = floor(kept / C * 2^32) with the quotient taken in fp64 (both operands are exact).
static uint32_t kept_to_thresh(uint64_t kept, uint64_t C) {
    return (uint32_t)std::floor((double)kept / (double)C * 4294967296.0);
}

void build_alias(const uint64_t* counts, uint32_t V, uint32_t* thresh, uint32_t* alias) {
    std::vector<double> weight(V);
    double wmax = 0.0;
    for (uint32_t i = 0; i < V; ++i) {
        double c = (double)(counts ? counts[i] : 1);
        double s = std::sqrt(std::sqrt(c));
        weight[i] = s * s * s;
        if (weight[i] > wmax) wmax = weight[i];
    }
    int e = 0;
    std::frexp(wmax, &e);                       // wmax = f * 2^e, 0.5 <= f < 1
    int log2V = 0;
    while ((1ull << log2V) < V) ++log2V;
    const int bits = 62 - log2V < 42 ? 62 - log2V : 42;
    std::vector<uint64_t> u(V);
    uint64_t total = 0;
    uint32_t biggest = 0;
    for (uint32_t i = 0; i < V; ++i) {
        u[i] = (uint64_t)std::floor(std::ldexp(weight[i], bits - e));
        total += u[i];
        if (u[i] > u[biggest]) biggest = i;     // first among equals
    }
    const uint64_t C = (total + V - 1) / V;
    u[biggest] += C * V - total;

    std::vector<uint32_t> light, heavy;
    for (uint32_t i = 0; i < V; ++i) {
        (u[i] < C ? light : heavy).push_back(i);
        thresh[i] = 0xFFFFFFFFu;
        alias[i] = i;
    }
    size_t li = 0, hi = 0;
    uint64_t r = u[heavy[0]];                   // the largest entry is never light
    for (;;) {
        if (r > C) {                            // top up the next light bucket
            const uint32_t l = light[li++];
            thresh[l] = kept_to_thresh(u[l], C);
            alias[l] = heavy[hi];
            r -= C - u[l];
        } else {                                // close the heavy entry's own bucket
            if (hi + 1 == heavy.size()) break;  // the last one keeps exactly C
            const uint32_t h = heavy[hi], next = heavy[hi + 1];
            if (r < C) {
                thresh[h] = kept_to_thresh(r, C);
                alias[h] = next;
            }
            r = u[next] - (C - r);
            ++hi;
        }
    }
}

inline uint32_t alias_draw(const uint32_t* thresh, const uint32_t* alias, uint32_t V, uint32_t ra, uint32_t rb) {
    uint32_t slot = mulhi32(ra, V);
    if (thresh[slot] == 0xFFFFFFFFu || rb < thresh[slot]) return slot;
    return alias[slot];
}

inline double sigmoid(double x) { return 1.0 / (1.0 + std::exp(-x)); }
// -log(sigmoid(x)) without overflow
inline double neg_log_sigmoid(double x) { return (x < 0 ? -x : 0.0) + std::log1p(std::exp(-std::fabs(x))); }

struct Message {
    std::vector<uint32_t> ids;     // ascending; [0,V) input rows, [V,2V) output rows
    std::vector<float> delta;      // ids.size() x d
    std::vector<uint64_t> g_snapshot;  // gradients the sender had applied when it computed this one
    int pending = 0;               // deliveries still outstanding
};

struct Delivery { uint64_t due, origin; uint32_t sender; };

struct LogRec { uint64_t origin, due, applied_at; uint32_t sender, staleness; };

struct Oracle {
    uint32_t V, d, window, k, batch, W, max_delay, reduction, max_grad_buffer = 1;
    float lr;
    uint64_t seed;
    std::vector<std::vector<float>> tin, tout;   // per replica V*d
    std::vector<uint64_t> counts;
    std::vector<uint32_t> thresh, alias;
    std::map<std::pair<uint32_t, uint64_t>, Message> msgs;   // (sender, step)
    std::vector<std::vector<Delivery>> inbox;                 // per receiver
    std::vector<std::set<uint64_t>> applied;                  // G_i, gradient id = step * W + sender
    std::vector<std::vector<LogRec>> log;                     // per receiver
    // taps of the last train_batch
    std::vector<uint32_t> last_neg;                           // P*k raw draws
    std::vector<double> last_g;                               // P*(1+k), masked -> 0
    uint32_t last_pairs = 0;
    std::pair<uint32_t, uint64_t> last_key{0, 0};
    std::vector<std::vector<Message>> buffered;               // per replica: gradients computed and not yet sent
};

uint32_t delay_of(const Oracle& o, uint64_t step, uint32_t sender, uint32_t receiver) {
    U4 c{{(uint32_t)step, sender, receiver, TAG_DELAY << 24}};
    U4 r = philox4x32_10(c, (uint32_t)o.seed, (uint32_t)(o.seed >> 32));
    return mulhi32(r.v[0], o.max_delay + 1);
}

void add_rows(Oracle& o, uint32_t replica, const Message& m) {
    const uint32_t d = o.d;
    for (size_t r = 0; r < m.ids.size(); ++r) {
        uint32_t id = m.ids[r];
        float* row = id < o.V ? &o.tin[replica][(size_t)id * d] : &o.tout[replica][(size_t)(id - o.V) * d];
        for (uint32_t e = 0; e < d; ++e) row[e] = row[e] + m.delta[r * d + e];
    }
}

uint32_t set_distance(const std::vector<uint64_t>& a_sorted, const std::set<uint64_t>& b) {
    size_t common = 0;
    for (uint64_t x : a_sorted) common += b.count(x);
    return (uint32_t)((a_sorted.size() + b.size() - common) - common);
}

void deliver(Oracle& o, uint32_t receiver, const Delivery& dl, uint64_t now) {
    auto key = std::make_pair(dl.sender, dl.origin);
    Message& m = o.msgs.at(key);
    uint32_t st = set_distance(m.g_snapshot, o.applied[receiver]);
    add_rows(o, receiver, m);
    o.applied[receiver].insert(dl.origin * o.W + dl.sender);
    o.log[receiver].push_back(LogRec{dl.origin, dl.due, now, dl.sender, st});
    if (--m.pending == 0 && key != o.last_key) o.msgs.erase(key);
}

}  // namespace

extern "C" {

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    U4 c{{ctr[0], ctr[1], ctr[2], ctr[3]}};
    U4 r = philox4x32_10(c, key[0], key[1]);
    for (int i = 0; i < 4; ++i) out[i] = r.v[i];
}

void orc_build_alias(const uint64_t* counts, uint32_t V, uint32_t* thresh, uint32_t* alias) {
    build_alias(counts, V, thresh, alias);
}

// Raw draw j of pair p of (replica, batch_index): one Philox call yields two draws.
uint32_t orc_negative(uint64_t seed, uint32_t replica, uint64_t batch_index, uint32_t p, uint32_t j,
                      const uint32_t* thresh, const uint32_t* alias, uint32_t V) {
    U4 c{{p, j >> 1, (uint32_t)batch_index, (TAG_NEGATIVE << 24) | replica}};
    U4 r = philox4x32_10(c, (uint32_t)seed, (uint32_t)(seed >> 32));
    return (j & 1) ? alias_draw(thresh, alias, V, r.v[2], r.v[3]) : alias_draw(thresh, alias, V, r.v[0], r.v[1]);
}

// Seeded initial input table: element e = row*d + col takes word (e & 3) of Philox(counter e >> 2).
void orc_init_input_table(uint64_t seed, uint32_t V, uint32_t d, float* dst) {
    const uint64_t n = (uint64_t)V * d;
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < (int64_t)n; ++e) {
        uint64_t blk = (uint64_t)e >> 2;
        U4 c{{(uint32_t)blk, (uint32_t)(blk >> 32), 0u, TAG_INIT << 24}};
        U4 r = philox4x32_10(c, (uint32_t)seed, (uint32_t)(seed >> 32));
        double u = ((double)(r.v[e & 3] >> 8) + 0.5) * (1.0 / 16777216.0);
        dst[e] = (float)((u - 0.5) / (double)d);
    }
}

Oracle* orc_create(uint32_t V, uint32_t d, uint32_t window, uint32_t k, uint32_t batch, uint32_t W,
                   float lr, uint32_t max_delay, uint64_t seed, uint32_t reduction, const uint64_t* counts,
                   const float* init_in, const float* init_out) {
    Oracle* o = new Oracle();
    o->V = V; o->d = d; o->window = window; o->k = k; o->batch = batch; o->W = W;
    o->lr = lr; o->max_delay = max_delay; o->seed = seed; o->reduction = reduction;
    const size_t n = (size_t)V * d;
    o->tin.assign(W, std::vector<float>());
    o->tout.assign(W, std::vector<float>());
    for (uint32_t r = 0; r < W; ++r) {
        o->tin[r].resize(n);
        o->tout[r].assign(n, 0.0f);
        if (init_in) std::memcpy(o->tin[r].data(), init_in, n * sizeof(float));
        else if (r == 0) orc_init_input_table(seed, V, d, o->tin[0].data());
        else o->tin[r] = o->tin[0];
        if (init_out) std::memcpy(o->tout[r].data(), init_out, n * sizeof(float));
    }
    o->counts.assign(V, 1);
    if (counts) std::copy(counts, counts + V, o->counts.begin());
    o->thresh.resize(V); o->alias.resize(V);
    build_alias(o->counts.data(), V, o->thresh.data(), o->alias.data());
    o->inbox.resize(W); o->applied.resize(W); o->log.resize(W); o->buffered.resize(W);
    return o;
}

void orc_destroy(Oracle* o) { delete o; }

// Rebuild the sampler table from the running counts (drift boundary).
void orc_update_sampler(Oracle* o) { build_alias(o->counts.data(), o->V, o->thresh.data(), o->alias.data()); }

void orc_get_sampler(Oracle* o, uint32_t* thresh, uint32_t* alias, uint64_t* counts) {
    if (thresh) std::copy(o->thresh.begin(), o->thresh.end(), thresh);
    if (alias) std::copy(o->alias.begin(), o->alias.end(), alias);
    if (counts) std::copy(o->counts.begin(), o->counts.end(), counts);
}

// The batch loss at the replica's current tables, with the draws of (replica, batch_index); changes
// nothing.  Used by the finite-difference pin.
double orc_batch_loss(Oracle* o, uint32_t replica, const int32_t* tokens, uint32_t n, uint64_t batch_index) {
    const uint32_t d = o->d, k = o->k, w = o->window;
    const float* tin = o->tin[replica].data();
    const float* tout = o->tout[replica].data();
    double loss = 0.0;
    uint32_t p = 0;
    for (uint32_t q = 0; q < n; ++q) {
        for (int64_t c = (int64_t)q - w; c <= (int64_t)q + w; ++c) {
            if (c < 0 || c >= (int64_t)n || c == (int64_t)q) continue;
            const float* v = tin + (size_t)tokens[q] * d;
            uint32_t ctx = (uint32_t)tokens[c];
            double x = 0.0;
            for (uint32_t e = 0; e < d; ++e) x += (double)tout[(size_t)ctx * d + e] * (double)v[e];
            loss += neg_log_sigmoid(x);
            for (uint32_t j = 0; j < k; ++j) {
                uint32_t r = orc_negative(o->seed, replica, batch_index, p, j, o->thresh.data(), o->alias.data(), o->V);
                if (r == ctx) continue;
                double y = 0.0;
                for (uint32_t e = 0; e < d; ++e) y += (double)tout[(size_t)r * d + e] * (double)v[e];
                loss += neg_log_sigmoid(-y);
            }
            ++p;
        }
    }
    return loss;
}

// The Model instance that trains the pairs whose centre word is `token` (Section 4.3: hash partitioner keyed by x).
uint32_t orc_route(uint64_t seed, uint32_t W, uint32_t token) {
    U4 c{{token, 0u, 0u, TAG_ROUTE << 24}};
    U4 r = philox4x32_10(c, (uint32_t)seed, (uint32_t)(seed >> 32));
    return mulhi32(r.v[0], W);
}

// Algorithm 1, train(), mini-batch branch.  Returns 0, or -1 when a token id is out of range (then
// nothing has changed).  n_rows_out (nullable) receives the message's row count.  routed: the replica
// trains only the pairs of the batch whose centre word is routed to it (taps of the other pairs: draws
// 0xFFFFFFFF, scalars 0).
static int train_batch(Oracle* o, uint32_t replica, const int32_t* tokens, uint32_t n, uint64_t batch_index,
                       double* loss_out, uint32_t* n_rows_out, bool routed) {
    const uint32_t V = o->V, d = o->d, k = o->k, w = o->window;
    if (replica >= o->W) return -2;
    for (uint32_t q = 0; q < n; ++q) if (tokens[q] < 0 || (uint32_t)tokens[q] >= V) return -1;
    auto mine = [&](uint32_t token) { return !routed || orc_route(o->seed, o->W, token) == replica; };
    for (uint32_t q = 0; q < n; ++q) if (mine((uint32_t)tokens[q])) o->counts[tokens[q]] += 1;

    // pairs in (centre position ascending, context offset ascending) order
    struct Pair { uint32_t centre, ctx; bool own; };
    std::vector<Pair> pairs;
    for (uint32_t q = 0; q < n; ++q)
        for (int64_t c = (int64_t)q - w; c <= (int64_t)q + w; ++c)
            if (c >= 0 && c < (int64_t)n && c != (int64_t)q)
                pairs.push_back(Pair{(uint32_t)tokens[q], (uint32_t)tokens[c], mine((uint32_t)tokens[q])});
    const size_t P = pairs.size();

    // negatives
    o->last_neg.assign(P * k, 0xFFFFFFFFu);
    for (size_t p = 0; p < P; ++p)
        for (uint32_t j = 0; j < k && pairs[p].own; ++j)
            o->last_neg[p * k + j] = orc_negative(o->seed, routed ? 0u : replica, batch_index, (uint32_t)p, j,
                                                  o->thresh.data(), o->alias.data(), V);

    // scalars at the snapshot
    const float* tin = o->tin[replica].data();
    const float* tout = o->tout[replica].data();
    const uint32_t K1 = k + 1;
    std::vector<double> g(P * K1, 0.0);
    std::vector<uint8_t> live(P * K1, 0);
    std::vector<double> pair_loss(P, 0.0);
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < (int64_t)P; ++p) {
        const float* v = tin + (size_t)pairs[p].centre * d;
        for (uint32_t j = 0; j < K1 && pairs[p].own; ++j) {
            uint32_t row = j == 0 ? pairs[p].ctx : o->last_neg[p * k + (j - 1)];
            if (j > 0 && row == pairs[p].ctx) continue;   // a negative equal to the positive is dropped
            const float* u = tout + (size_t)row * d;
            double x = 0.0;
            for (uint32_t e = 0; e < d; ++e) x += (double)u[e] * (double)v[e];
            if (j == 0) { g[p * K1] = sigmoid(x) - 1.0; pair_loss[p] += neg_log_sigmoid(x); }
            else { g[p * K1 + j] = sigmoid(x); pair_loss[p] += neg_log_sigmoid(-x); }
            live[p * K1 + j] = 1;
        }
    }
    double loss = 0.0;
    for (size_t p = 0; p < P; ++p) loss += pair_loss[p];
    o->last_g = g;
    o->last_pairs = (uint32_t)P;

    // every live (pair, j) term adds g*u to the centre's input row and g*v to the output row
    struct Term { uint32_t id; uint32_t src; double g; };   // id, src in the unified [0,2V) row space
    std::vector<Term> terms;
    terms.reserve(2 * P * K1);
    for (size_t p = 0; p < P; ++p)
        for (uint32_t j = 0; j < K1; ++j) {
            if (!live[p * K1 + j]) continue;
            uint32_t row = j == 0 ? pairs[p].ctx : o->last_neg[p * k + (j - 1)];
            terms.push_back(Term{pairs[p].centre, V + row, g[p * K1 + j]});
            terms.push_back(Term{V + row, pairs[p].centre, g[p * K1 + j]});
        }
    std::stable_sort(terms.begin(), terms.end(), [](const Term& a, const Term& b) { return a.id < b.id; });
    std::vector<size_t> seg;   // start of each distinct id
    for (size_t i = 0; i < terms.size(); ++i) if (i == 0 || terms[i].id != terms[i - 1].id) seg.push_back(i);
    const size_t U = seg.size();
    seg.push_back(terms.size());

    const double scale = o->reduction ? (double)o->lr / (double)P : (double)o->lr;
    Message m;
    m.ids.resize(U);
    m.delta.resize(U * d);
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t r = 0; r < (int64_t)U; ++r) {
        std::vector<double> sum(d, 0.0);
        for (size_t i = seg[r]; i < seg[r + 1]; ++i) {
            uint32_t s = terms[i].src;
            const float* src = s < V ? tin + (size_t)s * d : tout + (size_t)(s - V) * d;
            for (uint32_t e = 0; e < d; ++e) sum[e] += terms[i].g * (double)src[e];
        }
        m.ids[r] = terms[seg[r]].id;
        for (uint32_t e = 0; e < d; ++e) m.delta[r * d + e] = (float)(-scale * sum[e]);
    }

    // local apply (staleness 0)
    add_rows(*o, replica, m);
    if (loss_out) *loss_out = loss;
    if (n_rows_out) *n_rows_out = (uint32_t)U;
    // Algorithm 1, train, mini-batch branch: the gradient joins the buffer, and the buffer is sent once it
    // holds maxGradBuffer gradients.  The buffered gradients are summed row by row in the order they were computed (one fp32
    // addition per element and buffered gradient; a row missing from a gradient adds nothing), over
    // the union of their rows; the buffer is emptied after the send.
    o->buffered[replica].push_back(std::move(m));
    if (o->buffered[replica].size() < o->max_grad_buffer) return 0;
    {
        std::vector<Message>& buf = o->buffered[replica];
        if (buf.size() == 1) {
            m = std::move(buf[0]);
        } else {
            std::map<uint32_t, std::vector<float>> rows;
            for (const Message& b : buf)
                for (size_t r = 0; r < b.ids.size(); ++r) {
                    auto it = rows.find(b.ids[r]);
                    if (it == rows.end()) rows.emplace(b.ids[r], std::vector<float>(b.delta.begin() + r * d, b.delta.begin() + (r + 1) * d));
                    else for (uint32_t e = 0; e < d; ++e) it->second[e] = it->second[e] + b.delta[r * d + e];
                }
            m = Message();
            for (const auto& kv : rows) {
                m.ids.push_back(kv.first);
                m.delta.insert(m.delta.end(), kv.second.begin(), kv.second.end());
            }
        }
        buf.clear();
    }
    // send to every other replica
    m.g_snapshot.assign(o->applied[replica].begin(), o->applied[replica].end());
    o->applied[replica].insert(batch_index * o->W + replica);
    m.pending = (int)o->W - 1;
    auto key = std::make_pair(replica, batch_index);
    for (uint32_t j = 0; j < o->W; ++j)
        if (j != replica) o->inbox[j].push_back(Delivery{batch_index + delay_of(*o, batch_index, replica, j), batch_index, replica});
    // keep the newest message of this replica readable; drop the previous one if fully delivered
    auto prev = o->last_key;
    o->last_key = key;
    o->msgs[key] = std::move(m);
    auto it = o->msgs.find(prev);
    if (prev != key && it != o->msgs.end() && it->second.pending == 0) o->msgs.erase(it);
    return 0;
}

int orc_train_batch(Oracle* o, uint32_t replica, const int32_t* tokens, uint32_t n, uint64_t batch_index,
                    double* loss_out, uint32_t* n_rows_out) {
    return train_batch(o, replica, tokens, n, batch_index, loss_out, n_rows_out, false);
}
int orc_train_batch_routed(Oracle* o, uint32_t replica, const int32_t* tokens, uint32_t n, uint64_t batch_index,
                           double* loss_out, uint32_t* n_rows_out) {
    return train_batch(o, replica, tokens, n, batch_index, loss_out, n_rows_out, true);
}

void orc_set_max_grad_buffer(Oracle* o, uint32_t m) { o->max_grad_buffer = m < 1 ? 1 : m; }

// Algorithm 1, train(), gradient branch: every pending message for `replica` that is due at or
// before `step`, in (origin step, sender) order.  Returns how many were applied.
int orc_apply_messages(Oracle* o, uint32_t replica, uint64_t step) {
    auto& in = o->inbox[replica];
    std::vector<Delivery> due, rest;
    for (const Delivery& dl : in) (dl.due <= step ? due : rest).push_back(dl);
    std::sort(due.begin(), due.end(), [](const Delivery& a, const Delivery& b) {
        return a.origin != b.origin ? a.origin < b.origin : a.sender < b.sender; });
    for (const Delivery& dl : due) deliver(*o, replica, dl, step);
    in.swap(rest);
    return (int)due.size();
}

// End of run: everything still pending, per receiver in (due step, origin step, sender) order.
int orc_drain(Oracle* o) {
    int total = 0;
    for (uint32_t r = 0; r < o->W; ++r) {
        auto due = o->inbox[r];
        o->inbox[r].clear();
        std::sort(due.begin(), due.end(), [](const Delivery& a, const Delivery& b) {
            if (a.due != b.due) return a.due < b.due;
            return a.origin != b.origin ? a.origin < b.origin : a.sender < b.sender; });
        for (const Delivery& dl : due) deliver(*o, r, dl, dl.due);
        total += (int)due.size();
    }
    return total;
}

void orc_read_embeddings(Oracle* o, uint32_t replica, int which, uint32_t row0, uint32_t nrows, float* dst) {
    const std::vector<float>& t = which ? o->tout[replica] : o->tin[replica];
    std::memcpy(dst, t.data() + (size_t)row0 * o->d, (size_t)nrows * o->d * sizeof(float));
}

void orc_write_embeddings(Oracle* o, uint32_t replica, int which, uint32_t row0, uint32_t nrows, const float* src) {
    std::vector<float>& t = which ? o->tout[replica] : o->tin[replica];
    std::memcpy(t.data() + (size_t)row0 * o->d, src, (size_t)nrows * o->d * sizeof(float));
}

uint32_t orc_last_pairs(Oracle* o) { return o->last_pairs; }
void orc_read_negatives(Oracle* o, uint32_t* dst) { std::copy(o->last_neg.begin(), o->last_neg.end(), dst); }
void orc_read_g(Oracle* o, double* dst) { std::copy(o->last_g.begin(), o->last_g.end(), dst); }

// Message (replica, batch_index): returns its row count, or -1 when it is no longer held.
int64_t orc_read_message(Oracle* o, uint32_t replica, uint64_t batch_index, uint32_t* ids, float* delta) {
    auto it = o->msgs.find(std::make_pair(replica, batch_index));
    if (it == o->msgs.end()) return -1;
    const Message& m = it->second;
    if (ids) std::copy(m.ids.begin(), m.ids.end(), ids);
    if (delta) std::copy(m.delta.begin(), m.delta.end(), delta);
    return (int64_t)m.ids.size();
}

uint32_t orc_delay(Oracle* o, uint64_t step, uint32_t sender, uint32_t receiver) { return delay_of(*o, step, sender, receiver); }

// Delivery log of one receiver: records of 5 uint64 {origin step, sender, due step, applied at, staleness}.
uint64_t orc_log_size(Oracle* o, uint32_t replica) { return o->log[replica].size(); }
void orc_read_log(Oracle* o, uint32_t replica, uint64_t* dst) {
    for (const LogRec& r : o->log[replica]) {
        *dst++ = r.origin; *dst++ = r.sender; *dst++ = r.due; *dst++ = r.applied_at; *dst++ = r.staleness;
    }
}
uint64_t orc_pending(Oracle* o, uint32_t replica) { return o->inbox[replica].size(); }

// Event-level staleness bookkeeping on its own, for schedules that are not step-synchronous (the
// paper's Fig. 2 example).  A "book" holds the sets G_i; compute() snapshots G_i, applies the new
// gradient to i with staleness 0 and returns a gradient handle; apply() returns the staleness.
struct Book { std::vector<std::set<uint64_t>> G; std::vector<std::vector<uint64_t>> snap; };
Book* orc_book_create(uint32_t models) { Book* b = new Book(); b->G.resize(models); return b; }
void orc_book_destroy(Book* b) { delete b; }
uint64_t orc_book_compute(Book* b, uint32_t model) {
    uint64_t id = b->snap.size();
    b->snap.emplace_back(b->G[model].begin(), b->G[model].end());
    b->G[model].insert(id);
    return id;
}
uint32_t orc_book_apply(Book* b, uint32_t model, uint64_t grad) {
    uint32_t st = set_distance(b->snap[grad], b->G[model]);
    b->G[model].insert(grad);
    return st;
}
uint32_t orc_book_size(Book* b, uint32_t model) { return (uint32_t)b->G[model].size(); }

// Cosine difference 1 - cos(a_r, b_r) per row (the drift metric of Section 4.3, Table 1), fp64 arithmetic;
// two zero rows give 0, one zero row gives 1.
void orc_cosine_difference(const float* a, const float* b, uint32_t nrows, uint32_t d, float* out) {
    for (uint32_t r = 0; r < nrows; ++r) {
        double ab = 0.0, aa = 0.0, bb = 0.0;
        for (uint32_t e = 0; e < d; ++e) {
            const double x = a[(size_t)r * d + e], y = b[(size_t)r * d + e];
            ab += x * y; aa += x * x; bb += y * y;
        }
        double diff;
        if (aa == 0.0 && bb == 0.0) diff = 0.0;
        else if (aa == 0.0 || bb == 0.0) diff = 1.0;
        else diff = 1.0 - ab / (std::sqrt(aa) * std::sqrt(bb));
        out[r] = (float)diff;
    }
}

// The k rows that drifted most (largest cosine difference first, the smaller row id first among equal
// values), as Table 1 of Section 4.3 lists the words that moved most.  Values are ranked by the total
// order of their fp32 bit patterns (-NaN < -inf < ... < -0 < +0 < ... < +inf < +NaN), so the result is
// defined for every input.  Returns min(k, n), the number of entries written.
static uint32_t total_order_key(float x) {
    uint32_t b;
    std::memcpy(&b, &x, 4);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
uint32_t orc_top_drifted(const float* diff, uint32_t n, uint32_t k, uint32_t* ids, float* vals) {
    std::vector<uint32_t> order(n);
    for (uint32_t i = 0; i < n; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
        return total_order_key(diff[a]) > total_order_key(diff[b]);   // stable: equal values keep ascending ids
    });
    const uint32_t m = k < n ? k : n;
    for (uint32_t i = 0; i < m; ++i) {
        ids[i] = order[i];
        vals[i] = diff[order[i]];
    }
    return m;
}

int orc_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

}  // extern "C"
