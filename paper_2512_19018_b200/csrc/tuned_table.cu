// Persisted tuning table: shape class -> kernel family and knob values found by the offline sweep
// (`python -m paper_2512_19018_b200.tune --sweep`), the paper's performance evaluator (section 3.3: enumerate,
// prune, keep the best) made durable.  The table is a JSON file beside the library (tuned_sm100.json), read once
// on first use; the environment variable PEAK_TUNED_TABLE names another file, or switches the table off
// ("off", "0", "none").  Without a table, or for a shape no entry covers, the dispatcher's built-in rules
// apply; a knob set through peak_set_tuning always wins over the table.
//
// File format (everything else in the file is ignored):
//   {"entries": [ {"in": "bf16", "out": "bf16", "layout": "NN", "beta": 0, "M": 4096, "N": 4096, "K": 4096,
//                  "variant": "umma_2cta", "knobs": {"1": 512, "0": 16}}, ... ]}
// An entry covers problems of the same types, layout and beta class (zero / non-zero) whose M, N and K each
// lie within a factor sqrt(2) of the entry's.
#include <dlfcn.h>

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

#include "common.cuh"

namespace peak {
namespace {

struct Entry {
    int in = -1, out = -1, ta = 0, tb = 0, beta_nz = 0;
    int64_t M = 0, N = 0, K = 0;
    int variant = 0;  // 0 = dispatcher's choice
    int knob[PEAK_TUNE_COUNT_] = {};
};

// knobs a table may set: choices between equivalent kernels only, never test hooks or wait budgets
bool knob_allowed(int key) {
    switch (key) {
        case PEAK_TUNE_RASTER_GROUP: case PEAK_TUNE_TILE_N: case PEAK_TUNE_SPLIT_K: case PEAK_TUNE_EPILOGUE:
        case PEAK_TUNE_SGEMM_FMA: case PEAK_TUNE_TAIL_SPLIT: case PEAK_TUNE_SGEMM_COPY: case PEAK_TUNE_MULTICAST:
        case PEAK_TUNE_BALANCED_GRID: case PEAK_TUNE_EPILOGUE_WARPS: case PEAK_TUNE_K_ORDER: case PEAK_TUNE_SWAP_AB: case PEAK_TUNE_SGEMM_TRANSPOSE: case PEAK_TUNE_SHORT_A: case PEAK_TUNE_CLUSTER_K: case PEAK_TUNE_SHARE: case PEAK_TUNE_NARROW:
            return true;
    }
    return false;
}

// ---- a small JSON reader: objects, arrays, strings, numbers, true / false / null ---------------------------
struct Json {
    enum Kind { Null, Bool, Num, Str, Arr, Obj } kind = Null;
    double num = 0;
    std::string str;
    std::vector<Json> items;                              // array elements / object values
    std::vector<std::string> keys;                        // object keys (parallel to items)
    const Json *get(const char *k) const {
        if (kind != Obj) return nullptr;
        for (size_t i = 0; i < keys.size(); ++i)
            if (keys[i] == k) return &items[i];
        return nullptr;
    }
};
struct Reader {
    const char *p, *end;
    bool ok = true;
    int depth = 0;
    void ws() { while (p < end && (*p == ' ' || *p == '\n' || *p == '\t' || *p == '\r')) ++p; }
    bool lit(const char *s) {
        const size_t n = strlen(s);
        if ((size_t)(end - p) >= n && strncmp(p, s, n) == 0) { p += n; return true; }
        return false;
    }
    std::string string_() {
        std::string out;
        if (p >= end || *p != '"') { ok = false; return out; }
        ++p;
        while (p < end && *p != '"') {
            if (*p == '\\' && p + 1 < end) {
                ++p;
                switch (*p) {
                    case 'n': out += '\n'; break;
                    case 't': out += '\t'; break;
                    case 'u': out += '?'; p += (end - p > 4) ? 4 : 0; break;  // not needed for this file's fields
                    default: out += *p;
                }
                ++p;
            } else out += *p++;
        }
        if (p >= end) { ok = false; return out; }
        ++p;
        return out;
    }
    Json value() {
        Json j;
        ws();
        if (!ok || p >= end || ++depth > 32) { ok = false; return j; }
        if (*p == '{') {
            j.kind = Json::Obj;
            ++p; ws();
            if (p < end && *p == '}') { ++p; --depth; return j; }
            while (ok) {
                ws();
                std::string k = string_();
                ws();
                if (!ok || p >= end || *p != ':') { ok = false; break; }
                ++p;
                j.keys.push_back(k);
                j.items.push_back(value());
                ws();
                if (p < end && *p == ',') { ++p; continue; }
                if (p < end && *p == '}') { ++p; break; }
                ok = false;
            }
        } else if (*p == '[') {
            j.kind = Json::Arr;
            ++p; ws();
            if (p < end && *p == ']') { ++p; --depth; return j; }
            while (ok) {
                j.items.push_back(value());
                ws();
                if (p < end && *p == ',') { ++p; continue; }
                if (p < end && *p == ']') { ++p; break; }
                ok = false;
            }
        } else if (*p == '"') {
            j.kind = Json::Str;
            j.str = string_();
        } else if (lit("true")) { j.kind = Json::Bool; j.num = 1; }
        else if (lit("false")) { j.kind = Json::Bool; j.num = 0; }
        else if (lit("null")) { j.kind = Json::Null; }
        else {
            char *e = nullptr;
            j.kind = Json::Num;
            j.num = strtod(p, &e);
            if (e == p || e > end) ok = false; else p = e;
        }
        --depth;
        return j;
    }
};

int type_code(const std::string &s) {
    if (s == "f16") return (int)Elem::F16;
    if (s == "bf16") return (int)Elem::BF16;
    if (s == "f32") return (int)Elem::F32;
    if (s == "e4m3") return (int)Elem::E4M3;
    if (s == "e5m2") return (int)Elem::E5M2;
    return -1;
}
int variant_code(const std::string &s) {
    if (s == "umma_1cta") return PEAK_VARIANT_UMMA_1CTA;
    if (s == "umma_2cta") return PEAK_VARIANT_UMMA_2CTA;
    if (s == "sgemm") return PEAK_VARIANT_SGEMM;
    if (s == "fallback") return PEAK_VARIANT_FALLBACK;
    return 0;
}

struct Table {
    std::vector<Entry> entries;
    std::string path;
    bool loaded = false;
};
Table g_table;
std::mutex g_table_mutex;

// Parses `text`; entries with unknown types, a malformed layout or non-positive sizes are skipped.
// Returns the number of entries kept, or -1 when the text is not the JSON this reader understands.
int parse_table(const char *text, size_t len, std::vector<Entry> &out) {
    Reader r{text, text + len};
    Json root = r.value();
    r.ws();
    if (!r.ok || root.kind != Json::Obj) return -1;
    const Json *ents = root.get("entries");
    if (!ents || ents->kind != Json::Arr) return -1;
    for (const Json &e : ents->items) {
        if (e.kind != Json::Obj) continue;
        Entry t;
        const Json *in = e.get("in"), *o = e.get("out"), *lay = e.get("layout"), *M = e.get("M"), *N = e.get("N"),
                   *K = e.get("K"), *beta = e.get("beta"), *var = e.get("variant"), *kn = e.get("knobs");
        if (!in || !o || !lay || !M || !N || !K || in->kind != Json::Str || o->kind != Json::Str ||
            lay->kind != Json::Str || lay->str.size() != 2)
            continue;
        t.in = type_code(in->str); t.out = type_code(o->str);
        t.ta = lay->str[0] == 'T'; t.tb = lay->str[1] == 'T';
        t.M = (int64_t)M->num; t.N = (int64_t)N->num; t.K = (int64_t)K->num;
        t.beta_nz = (beta && beta->num != 0.0) ? 1 : 0;
        if (t.in < 0 || t.out < 0 || t.M < 1 || t.N < 1 || t.K < 1) continue;
        if (var && var->kind == Json::Str) t.variant = variant_code(var->str);
        if (kn && kn->kind == Json::Obj) {
            for (size_t i = 0; i < kn->keys.size(); ++i) {
                const int key = atoi(kn->keys[i].c_str());
                const double v = kn->items[i].num;
                if (kn->items[i].kind == Json::Num && key >= 0 && key < PEAK_TUNE_COUNT_ && knob_allowed(key) && v >= 0 &&
                    v < 1e6)
                    t.knob[key] = (int)v;
            }
        }
        out.push_back(t);
    }
    return (int)out.size();
}

int load_file(const char *path, std::vector<Entry> &out) {
    FILE *f = fopen(path, "rb");
    if (!f) return -2;
    std::string text;
    char buf[4096];
    size_t n;
    while ((n = fread(buf, 1, sizeof buf, f)) > 0 && text.size() < (8u << 20)) text.append(buf, n);
    fclose(f);
    return parse_table(text.data(), text.size(), out);
}

void ensure_loaded() {
    std::lock_guard<std::mutex> lock(g_table_mutex);
    if (g_table.loaded) return;
    g_table.loaded = true;
    const char *env = getenv("PEAK_TUNED_TABLE");
    std::string path;
    if (env && *env) {
        if (!strcmp(env, "off") || !strcmp(env, "0") || !strcmp(env, "none")) return;
        path = env;
    } else {
        Dl_info info;
        if (!dladdr(reinterpret_cast<void *>(&ensure_loaded), &info) || !info.dli_fname) return;
        path = info.dli_fname;
        const size_t slash = path.find_last_of('/');
        path = (slash == std::string::npos ? std::string(".") : path.substr(0, slash)) + "/tuned_sm100.json";
    }
    std::vector<Entry> ents;
    if (load_file(path.c_str(), ents) >= 0) {
        g_table.entries.swap(ents);
        g_table.path = path;
    }
}

bool near(int64_t x, int64_t ref) {  // within a factor sqrt(2) of the tuned size
    const double r = (double)x / (double)ref;
    return r >= 0.70710678 && r < 1.41421357;
}

thread_local const Entry *t_entry = nullptr;
thread_local Entry t_entry_copy;

}  // namespace

// ---- used by the dispatcher ------------------------------------------------------------------------------
TunedScope::TunedScope(const GemmArgs &g) {
    ensure_loaded();
    t_entry = nullptr;
    if (g.nbatch() > 1) return;
    std::lock_guard<std::mutex> lock(g_table_mutex);
    const int in = (int)in_elem(g.dtype), out = (int)out_elem(g.dtype);
    for (const Entry &e : g_table.entries) {
        if (e.in == in && e.out == out && e.ta == (g.transA ? 1 : 0) && e.tb == (g.transB ? 1 : 0) &&
            e.beta_nz == (g.beta != 0.0f ? 1 : 0) && near(g.M, e.M) && near(g.N, e.N) && near(g.K, e.K)) {
            t_entry_copy = e;  // a copy: the table may be reloaded by another thread
            t_entry = &t_entry_copy;
            return;
        }
    }
}
TunedScope::~TunedScope() { t_entry = nullptr; }

int tuned_knob(int key) { return (t_entry && key >= 0 && key < PEAK_TUNE_COUNT_) ? t_entry->knob[key] : 0; }
int tuned_variant() { return t_entry ? t_entry->variant : 0; }

}  // namespace peak

extern "C" {

int peak_tuned_table_load(const char *path) {
    using namespace peak;
    std::vector<Entry> ents;
    int n = 0;
    if (path && *path) {
        n = load_file(path, ents);
        if (n < 0) return n;  // -2: cannot open, -1: not understood; the current table stays
    }
    std::lock_guard<std::mutex> lock(g_table_mutex);
    g_table.loaded = true;
    g_table.entries.swap(ents);
    g_table.path = (path && *path) ? path : "";
    return n;
}

int peak_tuned_table_entries(void) {
    using namespace peak;
    ensure_loaded();
    std::lock_guard<std::mutex> lock(g_table_mutex);
    return (int)g_table.entries.size();
}

int peak_tuned_lookup(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float beta, int *variant,
                      int *knobs) {
    using namespace peak;
    if (dtype < PEAK_F16_F32 || dtype > PEAK_E5M2_F32 || M < 1 || N < 1 || K < 1) return 0;
    GemmArgs g{dtype, transA, transB, M, N, K, 1.0f, beta, nullptr, nullptr, nullptr, 0, 0, 0, nullptr};
    TunedScope scope(g);
    if (!t_entry) return 0;
    if (variant) *variant = t_entry->variant;
    if (knobs)
        for (int k = 0; k < PEAK_TUNE_COUNT_; ++k) knobs[k] = t_entry->knob[k];
    return 1;
}

}  // extern "C"
