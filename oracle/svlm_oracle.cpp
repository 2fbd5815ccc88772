// TEST INFRASTRUCTURE, NOT PRODUCT CODE.
//
// Plain, slow, fp64 CPU statement of the per-chunk KV-cache step of StreamingVLM's streaming
// inference (paper Section 2.1): the streaming-aware KV cache ("Streaming-aware KV Cache"
// paragraph), contiguous RoPE and contiguous 3D RoPE ("Contiguous RoPE" paragraph), and softmax
// attention of new tokens over the retained cache.  It exists so that the tests, the smoke check
// and the benchmark's CPU-baseline leg have something independent to compare the CUDA library
// with.  It shares no code with the CUDA library and must never be called from it.
//
// Everything is written as the definition, with no blocking, fusion or reordering:
//   * a stored token carries its stream ordinal gid, its type, its per-type ordinal ord, the
//     native position p the caller supplied, its current contiguous position c, and the amount a
//     by which it advanced the native position cursor;
//   * eviction keeps the first S text tokens (sinks), the last Tw text tokens and the last Vw
//     vision tokens, and left-shifts the position of every kept token by the native position span
//     freed by the evicted tokens that precede it;
//   * attention always rotates the *raw* keys at their current position (there is no incremental
//     re-rotation here), and a query sees every stored token whose gid does not exceed its own.
//
// Readings taken where the paper is silent are listed next to each step; the ones that are
// switches (sink_any_type, contiguous) keep the other reading testable.
//
// Parity pins (tests/test_oracle_*.py, CPU only): kept set and positions against a never-evicting
// brute force and a from-scratch 3D index assignment written separately in oracle/brute.py, window
// and sink invariants, the Figure-3 toy sizes worked by hand, closed-form rotation identities, and
// attention against a library softmax-attention routine in the no-eviction special case.
// Parity unpinned: the choice of readings itself (sinks are text tokens; append-then-evict order;
// the left-shift applied to a partially evicted vision block; native 3D index recipe; RoPE base):
// the paper prints no worked numbers for them.
//
// Build: g++ -O2 -fopenmp -shared -fPIC -o libsvlm_oracle.so svlm_oracle.cpp

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum { TEXT = 0, VISION = 1 };
enum { ROPE_1D = 0, ROPE_MROPE = 1 };

struct Token {
    int64_t gid;    // order of arrival in the stream, 0-based
    int type;       // TEXT or VISION
    int64_t ord;    // ordinal among tokens of the same type
    int64_t p[3];   // native position (t,h,w); 1D mode repeats the single index
    int64_t c[3];   // current contiguous position
    int64_t a;      // how far this token advanced the native position cursor
};

struct Oracle {
    int layers, kv_heads, head_dim;
    int64_t n_sink, vision_window, text_window;
    int rope_mode;
    double rope_base;
    int sections[3];
    int sink_any_type;   // 0: sinks are the first S TEXT tokens (default); 1: the first S tokens of any type
    int contiguous;      // 1: contiguous RoPE (default); 0: native RoPE (positions never shift)

    int64_t n_total = 0, n_text = 0, n_vis = 0, cursor = 0, shift_total = 0;
    std::vector<Token> stored;                      // stream order
    std::vector<std::vector<uint16_t>> kraw, vraw;  // per layer: [stored index][kv_head][dim] bf16 bits
    std::vector<std::vector<uint8_t>> has_kv;       // per layer: [stored index]
};

double widen_bf16(uint16_t bits) {
    uint32_t u = static_cast<uint32_t>(bits) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

// Which position axis rotates pair i (i in [0, d/2)): MRoPE gives the first sections[0] pairs to t,
// the next sections[1] to h and the rest to w; 1D uses a single index (stored in all three slots).
int axis_of_pair(const Oracle& o, int i) {
    if (o.rope_mode == ROPE_1D) return 0;
    if (i < o.sections[0]) return 0;
    if (i < o.sections[0] + o.sections[1]) return 1;
    return 2;
}

// R(c) x: pair (i, i + d/2) is rotated by the angle c_axis(i) * base^(-2i/d).
void rotate(const Oracle& o, const double* x, const int64_t c[3], double* y) {
    const int d = o.head_dim, half = d / 2;
    for (int i = 0; i < half; ++i) {
        const double theta = std::pow(o.rope_base, -2.0 * i / d);
        const double ang = static_cast<double>(c[axis_of_pair(o, i)]) * theta;
        const double cs = std::cos(ang), sn = std::sin(ang);
        y[i] = x[i] * cs - x[i + half] * sn;
        y[i + half] = x[i + half] * cs + x[i] * sn;
    }
}

// Retention rule of the streaming-aware KV cache, evaluated with the current per-type counts.
bool keep(const Oracle& o, const Token& t) {
    if (o.sink_any_type) {
        if (t.gid < o.n_sink) return true;
        if (t.type == TEXT) return t.ord >= o.n_text - o.text_window;
        return t.ord >= o.n_vis - o.vision_window;
    }
    if (t.type == TEXT) return t.ord < o.n_sink || t.ord >= o.n_text - o.text_window;
    return t.ord >= o.n_vis - o.vision_window;
}

}  // namespace

extern "C" {

void* svlmo_create(int layers, int kv_heads, int head_dim, int64_t n_sink, int64_t vision_window,
                   int64_t text_window, int rope_mode, double rope_base, const int* sections,
                   int sink_any_type, int contiguous) {
    Oracle* o = new Oracle;
    o->layers = layers; o->kv_heads = kv_heads; o->head_dim = head_dim;
    o->n_sink = n_sink; o->vision_window = vision_window; o->text_window = text_window;
    o->rope_mode = rope_mode; o->rope_base = rope_base;
    for (int k = 0; k < 3; ++k) o->sections[k] = sections ? sections[k] : 0;
    o->sink_any_type = sink_any_type; o->contiguous = contiguous;
    o->kraw.resize(layers); o->vraw.resize(layers); o->has_kv.resize(layers);
    return o;
}

void svlmo_destroy(void* h) { delete static_cast<Oracle*>(h); }

// Append n tokens in stream order.  K and V are bf16 bit patterns [layers][n][kv_heads][head_dim]
// (un-rotated) or null when only the metadata is being followed (values can be supplied later
// with svlmo_set_kv).  pos is [n] in 1D mode and [n][3] in MRoPE mode.
void svlmo_append(void* h, const uint16_t* K, const uint16_t* V, const uint8_t* types,
                  const int32_t* pos, int64_t n) {
    Oracle& o = *static_cast<Oracle*>(h);
    const size_t row = static_cast<size_t>(o.kv_heads) * o.head_dim;
    for (int64_t i = 0; i < n; ++i) {
        Token t;
        t.gid = o.n_total++;
        t.type = types[i];
        t.ord = (t.type == TEXT) ? o.n_text++ : o.n_vis++;
        for (int k = 0; k < 3; ++k)
            t.p[k] = (o.rope_mode == ROPE_1D) ? pos[i] : pos[3 * i + k];
        const int64_t top = std::max(t.p[0], std::max(t.p[1], t.p[2])) + 1;
        t.a = std::max<int64_t>(0, top - o.cursor);
        o.cursor += t.a;
        for (int k = 0; k < 3; ++k) t.c[k] = t.p[k] - o.shift_total;
        o.stored.push_back(t);
        for (int l = 0; l < o.layers; ++l) {
            const size_t at = o.kraw[l].size();
            o.kraw[l].resize(at + row, 0);
            o.vraw[l].resize(at + row, 0);
            if (K && V) {
                const size_t src = (static_cast<size_t>(l) * n + i) * row;
                std::memcpy(&o.kraw[l][at], K + src, row * sizeof(uint16_t));
                std::memcpy(&o.vraw[l][at], V + src, row * sizeof(uint16_t));
            }
            o.has_kv[l].push_back(K && V ? 1 : 0);
        }
    }
}

// Supply raw K/V of one layer for stored tokens named by gid (tokens no longer stored are skipped).
// K, V: [n][kv_heads][head_dim] bf16 bits.
void svlmo_set_kv(void* h, int layer, const int64_t* gids, const uint16_t* K, const uint16_t* V, int64_t n) {
    Oracle& o = *static_cast<Oracle*>(h);
    const size_t row = static_cast<size_t>(o.kv_heads) * o.head_dim;
    for (int64_t i = 0; i < n; ++i) {
        auto it = std::lower_bound(o.stored.begin(), o.stored.end(), gids[i],
                                   [](const Token& t, int64_t g) { return t.gid < g; });
        if (it == o.stored.end() || it->gid != gids[i]) continue;
        const size_t idx = static_cast<size_t>(it - o.stored.begin());
        std::memcpy(&o.kraw[layer][idx * row], K + i * row, row * sizeof(uint16_t));
        std::memcpy(&o.vraw[layer][idx * row], V + i * row, row * sizeof(uint16_t));
        o.has_kv[layer][idx] = 1;
    }
}

// Evict, compact and re-index.  Every kept token moves left by the native span (sum of a) of the
// evicted tokens before it, so positions stay contiguous with the last retained token; tokens that
// arrive later are shifted by the running total.
void svlmo_evict(void* h) {
    Oracle& o = *static_cast<Oracle*>(h);
    const size_t row = static_cast<size_t>(o.kv_heads) * o.head_dim;
    std::vector<Token> kept;
    std::vector<std::vector<uint16_t>> k2(o.layers), v2(o.layers);
    std::vector<std::vector<uint8_t>> f2(o.layers);
    int64_t freed = 0;  // E(i): span freed by evicted tokens before the current one
    for (size_t idx = 0; idx < o.stored.size(); ++idx) {
        Token t = o.stored[idx];
        if (!keep(o, t)) {
            if (o.contiguous) freed += t.a;
            continue;
        }
        for (int k = 0; k < 3; ++k) t.c[k] -= freed;
        kept.push_back(t);
        for (int l = 0; l < o.layers; ++l) {
            k2[l].insert(k2[l].end(), o.kraw[l].begin() + idx * row, o.kraw[l].begin() + (idx + 1) * row);
            v2[l].insert(v2[l].end(), o.vraw[l].begin() + idx * row, o.vraw[l].begin() + (idx + 1) * row);
            f2[l].push_back(o.has_kv[l][idx]);
        }
    }
    o.shift_total += freed;
    o.stored.swap(kept);
    o.kraw.swap(k2); o.vraw.swap(v2); o.has_kv.swap(f2);
}

int64_t svlmo_count(void* h) { return static_cast<int64_t>(static_cast<Oracle*>(h)->stored.size()); }

// Stored tokens in stream order.  Any output pointer may be null.  counters: n_total, n_text,
// n_vis, cursor, shift_total.
void svlmo_query(void* h, int64_t* gids, int32_t* pos3, uint8_t* types, int64_t* advances, int64_t* counters) {
    Oracle& o = *static_cast<Oracle*>(h);
    for (size_t i = 0; i < o.stored.size(); ++i) {
        if (gids) gids[i] = o.stored[i].gid;
        if (types) types[i] = static_cast<uint8_t>(o.stored[i].type);
        if (advances) advances[i] = o.stored[i].a;
        if (pos3) for (int k = 0; k < 3; ++k) pos3[3 * i + k] = static_cast<int32_t>(o.stored[i].c[k]);
    }
    if (counters) {
        counters[0] = o.n_total; counters[1] = o.n_text; counters[2] = o.n_vis;
        counters[3] = o.cursor; counters[4] = o.shift_total;
    }
}

// R(c) x for one head row in fp64 (exposed for the rotation-identity pins).
void svlmo_rotate(void* h, const double* x, const int64_t* c3, double* y) {
    rotate(*static_cast<Oracle*>(h), x, c3, y);
}

// Keys of one layer rotated at their current positions: out is fp64 [stored][kv_heads][head_dim].
void svlmo_rotated_k(void* h, int layer, double* out) {
    Oracle& o = *static_cast<Oracle*>(h);
    const int d = o.head_dim;
    const size_t row = static_cast<size_t>(o.kv_heads) * d;
    std::vector<double> x(d);
    for (size_t j = 0; j < o.stored.size(); ++j)
        for (int g = 0; g < o.kv_heads; ++g) {
            for (int e = 0; e < d; ++e) x[e] = widen_bf16(o.kraw[layer][j * row + g * d + e]);
            rotate(o, x.data(), o.stored[j].c, out + j * row + g * d);
        }
}

// Raw values of one layer widened to fp64: out is [stored][kv_heads][head_dim].
void svlmo_values(void* h, int layer, double* out) {
    Oracle& o = *static_cast<Oracle*>(h);
    const size_t n = o.stored.size() * static_cast<size_t>(o.kv_heads) * o.head_dim;
    for (size_t i = 0; i < n; ++i) out[i] = widen_bf16(o.vraw[layer][i]);
}

// Attention of the last n_q appended tokens over the stored tokens of one layer.
//   Q      bf16 bits [n_q][q_heads][head_dim], un-rotated
//   q_pos  native positions of the queries ([n_q] or [n_q][3])
//   rows   which query rows to compute (null: all n_q); n_rows entries
//   out    fp64 [n_rows][q_heads][head_dim]
// Query row r has gid n_total - n_q + r, is rotated at q_pos - shift_total, and sees stored tokens
// with gid <= its own; query head hq reads KV head hq / (q_heads / kv_heads); scores are scaled by
// 1/sqrt(head_dim); softmax subtracts the row maximum; an empty visible set gives zeros.
// Returns 0, or -1 if a visible token of this layer never received K/V values.
int svlmo_attend(void* h, int layer, const uint16_t* Q, const int32_t* q_pos, int64_t n_q, int q_heads,
                 const int64_t* rows, int64_t n_rows, double* out) {
    Oracle& o = *static_cast<Oracle*>(h);
    const int d = o.head_dim;
    const int group = q_heads / o.kv_heads;
    const size_t row = static_cast<size_t>(o.kv_heads) * d;
    const size_t n_st = o.stored.size();
    if (!rows) n_rows = n_q;

    std::vector<double> krot(n_st * row), vals(n_st * row);
    svlmo_rotated_k(h, layer, krot.data());
    svlmo_values(h, layer, vals.data());
    const double scale = 1.0 / std::sqrt(static_cast<double>(d));
    int missing = 0;

#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int64_t rr = 0; rr < n_rows; ++rr) {
        for (int hq = 0; hq < q_heads; ++hq) {
            const int64_t r = rows ? rows[rr] : rr;
            const int64_t gid_q = o.n_total - n_q + r;
            int64_t cq[3];
            for (int k = 0; k < 3; ++k)
                cq[k] = ((o.rope_mode == ROPE_1D) ? q_pos[r] : q_pos[3 * r + k]) - o.shift_total;
            std::vector<double> x(d), qr(d), s(n_st);
            for (int e = 0; e < d; ++e) x[e] = widen_bf16(Q[(static_cast<size_t>(r) * q_heads + hq) * d + e]);
            rotate(o, x.data(), cq, qr.data());
            const int g = hq / group;
            double m = -std::numeric_limits<double>::infinity();
            size_t n_vis = 0;
            for (size_t j = 0; j < n_st; ++j) {
                if (o.stored[j].gid > gid_q) break;   // stored is in stream order
                if (!o.has_kv[layer][j]) {
#pragma omp atomic write
                    missing = 1;
                }
                double acc = 0.0;
                const double* kj = &krot[j * row + g * d];
                for (int e = 0; e < d; ++e) acc += qr[e] * kj[e];
                s[j] = acc * scale;
                m = std::max(m, s[j]);
                n_vis = j + 1;
            }
            double* y = out + (static_cast<size_t>(rr) * q_heads + hq) * d;
            for (int e = 0; e < d; ++e) y[e] = 0.0;
            if (n_vis == 0) continue;
            double denom = 0.0;
            for (size_t j = 0; j < n_vis; ++j) { s[j] = std::exp(s[j] - m); denom += s[j]; }
            for (size_t j = 0; j < n_vis; ++j) {
                const double w = s[j] / denom;
                const double* vj = &vals[j * row + g * d];
                for (int e = 0; e < d; ++e) y[e] += w * vj[e];
            }
        }
    }
    return missing ? -1 : 0;
}

int svlmo_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}

}  // extern "C"
