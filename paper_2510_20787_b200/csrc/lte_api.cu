// C-ABI entry points of liblte: argument validation and dispatch.  No torch types, no allocation.
#include <math.h>

#include <atomic>

#include "common.cuh"

namespace lte {

int launch_prefill_tc(const Params& p, const void* q, const void* k, const void* v, const int32_t* idx,
                      const int32_t* cnt, void* o, float* lse, void* ws, size_t ws_bytes, cudaStream_t st,
                      const int32_t* leave = nullptr);
int prefill_status_fetch_and_clear();
int decode_status_fetch_and_clear();
int scores_status_fetch_and_clear();
int stack_tc_status_fetch_and_clear();
int stack_bwd_tc_status_fetch_and_clear();
int bwd_status_fetch_and_clear();
int decode_tc_status_fetch_and_clear();

// SM count of the current device, looked up once per device
int device_sm_count(int* n_sm)
{
    static PerDevice<int> table;
    return table.get(n_sm, [](int* out) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(out, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || *out <= 0)
            return (int)LTE_ERR_CUDA;
        return (int)LTE_OK;
    });
}

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(const lte_shape* s, bool need_T)
{
    if (!s) return LTE_ERR_INVALID_ARG;
    if (s->B <= 0 || s->H <= 0 || s->W <= 0 || s->R < 0 || s->sink < 0 || s->group < 0) return LTE_ERR_INVALID_ARG;
    if (need_T ? s->T <= 0 : s->T < 0) return LTE_ERR_INVALID_ARG;
    if (s->dtype != LTE_F32 && s->dtype != LTE_BF16) return LTE_ERR_INVALID_ARG;
    if (s->d != 32 && s->d != 64 && s->d != 128) return LTE_ERR_UNSUPPORTED;
    if (!(s->tau < 1.0f)) return LTE_ERR_INVALID_ARG;
    if ((double)s->B * s->H * (s->group > 1 ? s->group : 1) * (double)(s->T > 0 ? s->T : 1) * s->d > 2.0e10) return LTE_ERR_UNSUPPORTED;
    return LTE_OK;
}

int check_conv(const lte_shape* s, const lte_conv* c)
{
    if (!c || !c->w) return LTE_ERR_INVALID_ARG;
    if (c->n_layers != 1 || c->dilation != 1) return LTE_ERR_UNSUPPORTED;
    if (c->kernel < 1 || c->kernel > kMaxTaps || (c->kernel & 1) == 0) return LTE_ERR_INVALID_ARG;
    if (s->W < c->kernel) return LTE_ERR_INVALID_ARG;     // the receptive field must fit in the window
    return LTE_OK;
}

Params make_params(const lte_shape* s, const lte_conv* c)
{
    Params p;
    p.B = s->B; p.H = s->H; p.T = s->T; p.d = s->d; p.W = s->W; p.R = s->R; p.sink = s->sink;
    p.G = s->group > 1 ? s->group : 1;
    p.K = c ? c->kernel : 1; p.half = p.K / 2;
    p.stack = 0;
    p.qoff = 0;
    if (c && c->n_layers == 3) { p.stack = 1; p.K = 13; p.half = 6; }   // the paper's stack: receptive field 13
    p.zthr = s->tau <= 0.f ? -INFINITY : (float)(log((double)s->tau) - log1p(-(double)s->tau));
    p.scale = s->softmax_scale > 0.f ? s->softmax_scale : (float)(1.0 / sqrt((double)s->d));
    p.dtype = s->dtype;
    p.w = c ? c->w : nullptr;
    p.bias = c ? c->bias : nullptr;
    return p;
}

// the single layer, or the paper's stack where the decode cache takes it (d = 32 or 64, window at least 20 tokens: the
// ring has to hold a token's receptive field of 13 with room for a scoring period)
int check_conv_or_stack(const lte_shape* s, const lte_conv* c)
{
    if (c && c->w && c->n_layers == 3) {
        if (c->kernel != 3 || c->dilation != 2 || (s->d != 32 && s->d != 64)) return LTE_ERR_UNSUPPORTED;
        if (s->W < 20 || !aligned16(c->w)) return LTE_ERR_INVALID_ARG;
        return LTE_OK;
    }
    return check_conv(s, c);
}

int check_arch()
{
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return LTE_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return LTE_ERR_CUDA;
    return major == 10 ? LTE_OK : LTE_ERR_ARCH;
}

// scratch of lte_cache_score: the ring in time order (keys, values), its logits, the tensor-core scorer's weight image
struct CacheScorePlan { size_t klin, vlin, zlin, tc, total; };
CacheScorePlan cache_score_plan(const lte_shape* s, const lte_conv* c)
{
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    CacheScorePlan w;
    const size_t rows = (size_t)s->B * s->H * s->W, esz = s->dtype == LTE_BF16 ? 2 : 4;
    size_t off = 0;
    w.klin = off; off += up(rows * s->d * esz);
    w.vlin = off; off += up(rows * s->d * esz);
    w.zlin = off; off += up(rows * 4);
    w.tc = off;
    lte_shape s2 = *s; s2.T = s->W;
    off += up(scores_stack_tc_workspace(make_params(&s2, c)));
    w.total = off;
    return w;
}

// scratch of lte_attn_prefill_chunk, sized for the longest local sequence (pool rows + full ring + chunk)
struct ChunkPlan { size_t klin, vlin, z, zrank, zsrc, oldpos, idx, cnt, gate, ulist, leave, ucnt, sub, att, total; int ucap; };
ChunkPlan chunk_plan(const lte_shape* s, const lte_conv* c, bool streaming = false)
{
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    ChunkPlan w;
    const size_t bhk = (size_t)s->B * s->H;
    const size_t Tm = (size_t)s->R + s->W + s->T, esz = s->dtype == LTE_BF16 ? 2 : 4;
    size_t off = 0;
    w.klin = off; off += up(bhk * Tm * s->d * esz);
    w.vlin = off; off += up(bhk * Tm * s->d * esz);
    w.z = off; off += up(bhk * Tm * 4);
    w.zrank = off; off += up(bhk * Tm * 4);
    w.zsrc = off; off += up(bhk * ((size_t)s->R + s->W) * 4);
    w.oldpos = off; off += up(bhk * (size_t)(s->R > 0 ? s->R : 1) * 4);
    w.idx = off; off += up(bhk * (size_t)(s->R > 0 ? s->R : 1) * 4);
    w.cnt = off; off += up(bhk * 4);
    w.gate = off; off += up(bhk * 4);                        // per head: the cache held n_past tokens (written by every call's gather)
    // streaming reading: every entry that is in the pool at some query of the chunk (at most the old pool plus one per
    // token that leaves the window), and the query from which each is gone
    w.ucap = s->R + s->T;
    w.ulist = w.leave = w.ucnt = off;
    if (streaming) {
        w.ulist = off; off += up(bhk * (size_t)w.ucap * 4);
        w.leave = off; off += up(bhk * (size_t)w.ucap * 4);
        w.ucnt = off; off += up(bhk * 4);
    }
    w.sub = off;
    if (c && c->n_layers == 3) {
        lte_shape s2 = *s; s2.T = (int32_t)Tm;
        off += up(scores_stack_tc_workspace(make_params(&s2, c)));
    }
    w.att = off;                                             // the attention's compacted retained rows (streaming: of the entry list)
    {
        Params pa = make_params(s, c);
        if (streaming) pa.R = w.ucap;
        off += up(prefill_compact_bytes(pa));
    }
    w.total = off;
    return w;
}

}  // namespace
}  // namespace lte

using namespace lte;

extern "C" {

const char* lte_strerror(int status)
{
    switch (status) {
        case LTE_OK: return "ok";
        case LTE_ERR_INVALID_ARG: return "invalid argument";
        case LTE_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case LTE_ERR_WORKSPACE: return "workspace too small";
        case LTE_ERR_CUDA: return "CUDA call failed";
        case LTE_ERR_ARCH: return "device is not compute capability 10.x";
        case LTE_ERR_DEVICE_STATUS: return "a kernel recorded an anomaly";
    }
    return "unknown status";
}

int lte_device_status(void)
{
    const int h = prefill_status_fetch_and_clear();
    const int g = decode_status_fetch_and_clear();
    const int f = scores_status_fetch_and_clear();
    const int b = bwd_status_fetch_and_clear();
    const int d = decode_tc_status_fetch_and_clear();
    const int t = stack_tc_status_fetch_and_clear();
    const int u = stack_bwd_tc_status_fetch_and_clear();
    const int k = chunk_status_fetch_and_clear();
    if (h < 0 || g < 0 || f < 0 || b < 0 || d < 0 || t < 0 || u < 0 || k < 0) return LTE_ERR_CUDA;
    return (h == 0 && g == 0 && f == 0 && b == 0 && d == 0 && t == 0 && u == 0 && k == 0) ? LTE_OK : LTE_ERR_DEVICE_STATUS;
}

size_t lte_workspace_bytes(int op, const lte_shape* s, const lte_conv* c)
{
    if (!s) return 0;
    if (op == LTE_OP_BWD) {
        if (check_shape(s, true) != LTE_OK || !c) return 0;
        Params p = make_params(s, c);
        return bwd_workspace_bytes(p, LTE_BWD_CNN_INPUT_GRAD);
    }
    if (op == LTE_OP_DECODE && c && c->n_layers == 3) {
        if (check_shape(s, false) != LTE_OK) return 0;
        return cache_score_plan(s, c).total;
    }
    if (op == LTE_OP_PREFILL) {
        if (check_shape(s, true) != LTE_OK) return 0;
        return prefill_compact_bytes(make_params(s, nullptr));
    }
    if (op == LTE_OP_STATS) {
        if (check_shape(s, true) != LTE_OK) return 0;
        return ((size_t)s->B * s->H * 2 * sizeof(float) + 255) / 256 * 256;
    }
    if (op == LTE_OP_CHUNK || op == LTE_OP_CHUNK_STREAM) {
        if (check_shape(s, true) != LTE_OK || !c) return 0;
        if ((double)s->B * s->H * (s->group > 1 ? s->group : 1) * ((double)s->R + s->W + s->T) * s->d > 2.0e10) return 0;
        return chunk_plan(s, c, op == LTE_OP_CHUNK_STREAM).total;
    }
    if (op == LTE_OP_SCORES && c && c->n_layers == 3) {
        if (check_shape(s, true) != LTE_OK) return 0;
        return scores_stack_tc_workspace(make_params(s, c));
    }
    return 0;
}

int lte_scores(const lte_shape* s, const lte_conv* c, const void* k, const void* v, float* z, float* r_or_null,
               void* ws, size_t ws_bytes, void* stream)
{
    int e = check_shape(s, true); if (e) return e;
    if (c && c->w && c->n_layers == 3) {
        // the paper's stack: kernel 3, dilation 2, channels 2d -> d -> d/2 -> d/4 -> 1 (packed parameters, see lte.h)
        if (c->kernel != 3 || c->dilation != 2) return LTE_ERR_UNSUPPORTED;
        if (s->d != 32 && s->d != 64) return LTE_ERR_UNSUPPORTED;
        if (s->W < 7) return LTE_ERR_INVALID_ARG;            // tokens must be scored before they leave the window
        if (!k || !v || !z || !aligned16(k) || !aligned16(v) || !aligned16(c->w)) return LTE_ERR_INVALID_ARG;
        e = check_arch(); if (e) return e;
        Params p = make_params(s, c);
        // tensor cores where the shape allows and the caller brought the workspace for the split weight image
        e = launch_scores_stack_tc(p, k, v, z, r_or_null, ws, ws_bytes, (cudaStream_t)stream);
        if (e != LTE_ERR_UNSUPPORTED) return e;
        return launch_scores_stack(p, k, v, z, r_or_null, (cudaStream_t)stream);
    }
    e = check_conv(s, c); if (e) return e;
    if (!k || !v || !z || !aligned16(k) || !aligned16(v)) return LTE_ERR_INVALID_ARG;
    e = check_arch(); if (e) return e;
    return launch_scores(make_params(s, c), k, v, z, r_or_null, (cudaStream_t)stream);
}

int lte_select(const lte_shape* s, const float* z, int32_t* idx, int32_t* cnt, int32_t* ncand_or_null, void* ws,
               size_t ws_bytes, void* stream)
{
    (void)ws; (void)ws_bytes;
    int e = check_shape(s, true); if (e) return e;
    if (!z || !cnt || (s->R > 0 && !idx)) return LTE_ERR_INVALID_ARG;
    if (s->T - s->W > (1 << 24)) return LTE_ERR_UNSUPPORTED;
    e = check_arch(); if (e) return e;
    return launch_select(make_params(s, nullptr), z, idx, cnt, ncand_or_null, (cudaStream_t)stream);
}

int lte_select_rule(const lte_shape* s, int rule, const float* score, int32_t* idx, int32_t* cnt, int32_t* ncand_or_null,
                    void* ws, size_t ws_bytes, void* stream)
{
    if (rule == LTE_RULE_LEARNED) return lte_select(s, score, idx, cnt, ncand_or_null, ws, ws_bytes, stream);
    int e = check_shape(s, true); if (e) return e;
    if (!cnt || (s->R > 0 && !idx)) return LTE_ERR_INVALID_ARG;
    if (s->T - s->W > (1 << 24)) return LTE_ERR_UNSUPPORTED;
    if (rule == LTE_RULE_UNIFORM) {
        e = check_arch(); if (e) return e;
        return launch_select_uniform(make_params(s, nullptr), idx, cnt, ncand_or_null, (cudaStream_t)stream);
    }
    if (rule == LTE_RULE_ACCUM_ATTN) {                       // the learned rule's ranking without its threshold
        if (!score) return LTE_ERR_INVALID_ARG;
        e = check_arch(); if (e) return e;
        Params p = make_params(s, nullptr);
        p.zthr = -INFINITY;
        return launch_select(p, score, idx, cnt, ncand_or_null, (cudaStream_t)stream);
    }
    return LTE_ERR_INVALID_ARG;
}

int lte_attn_colsum(const lte_shape* s, const void* q, const void* k, const float* lse, const int32_t* idx, const int32_t* cnt,
                    float* a, void* stream)
{
    int e = check_shape(s, true); if (e) return e;
    if (!q || !k || !lse || !cnt || (s->R > 0 && !idx) || !a) return LTE_ERR_INVALID_ARG;
    e = check_arch(); if (e) return e;
    return launch_colsum(make_params(s, nullptr), q, k, lse, idx, cnt, a, (cudaStream_t)stream);
}

int lte_attn_prefill(const lte_shape* s, const void* q, const void* k, const void* v, const int32_t* idx,
                     const int32_t* cnt, void* o, float* lse, void* ws, size_t ws_bytes, void* stream)
{
    int e = check_shape(s, true); if (e) return e;
    if (!q || !k || !v || !o || !lse || !cnt || (s->R > 0 && !idx)) return LTE_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return LTE_ERR_INVALID_ARG;
    e = check_arch(); if (e) return e;
    Params p = make_params(s, nullptr);
    if (s->dtype == LTE_BF16) return launch_prefill_tc(p, q, k, v, idx, cnt, o, lse, ws, ws_bytes, (cudaStream_t)stream);
    return launch_prefill_simt(p, q, k, v, idx, cnt, o, lse, (cudaStream_t)stream);
}

size_t lte_cache_bytes(const lte_shape* s)
{
    if (!s || s->B <= 0 || s->H <= 0 || s->W <= 0 || s->R < 0 || s->d <= 0) return 0;
    const CacheLayout L = cache_layout(s->d, s->W, s->R, s->dtype);
    return L.header + (size_t)s->B * s->H * L.stride;
}

int lte_cache_init(const lte_shape* s, const lte_conv* c, const void* k, const void* v, const float* z,
                   const int32_t* idx, const int32_t* cnt, void* cache, void* stream)
{
    int e = check_shape(s, false); if (e) return e;
    e = check_conv_or_stack(s, c); if (e) return e;
    if (!cache || !aligned16(cache)) return LTE_ERR_INVALID_ARG;
    if (s->T > 0 && (!k || !v || !z || !cnt || (s->R > 0 && !idx))) return LTE_ERR_INVALID_ARG;
    e = check_arch(); if (e) return e;
    return launch_cache_init(make_params(s, c), k, v, z, idx, cnt, cache, (cudaStream_t)stream);
}

int lte_cache_score(const lte_shape* s, const lte_conv* c, void* cache, void* ws, size_t ws_bytes, void* stream)
{
    return lte_cache_score_unrope(s, c, cache, nullptr, nullptr, 0, ws, ws_bytes, stream);
}

int lte_cache_score_unrope(const lte_shape* s, const lte_conv* c, void* cache, const float* rope_cos, const float* rope_sin,
                           int32_t rope_len, void* ws, size_t ws_bytes, void* stream)
{
    int e = check_shape(s, false); if (e) return e;
    if ((rope_cos == nullptr) != (rope_sin == nullptr) || (rope_cos && rope_len <= 0)) return LTE_ERR_INVALID_ARG;
    if (!c || !c->w || c->n_layers != 3) return LTE_ERR_UNSUPPORTED;       // the single layer is scored inside the step
    e = check_conv_or_stack(s, c); if (e) return e;
    if (!cache || !aligned16(cache)) return LTE_ERR_INVALID_ARG;
    const CacheScorePlan w = cache_score_plan(s, c);
    if (!ws || ((uintptr_t)ws & 255u) != 0 || ws_bytes < w.total) return LTE_ERR_WORKSPACE;
    e = check_arch(); if (e) return e;
    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)ws;
    lte_shape s2 = *s; s2.T = s->W;                                         // the ring as a W-token sequence
    Params p = make_params(&s2, c);
    e = launch_ring_linearize(p, cache, base + w.klin, base + w.vlin, rope_cos, rope_sin, rope_len, st); if (e) return e;
    float* zlin = (float*)(base + w.zlin);
    e = launch_scores_stack_tc(p, base + w.klin, base + w.vlin, zlin, nullptr, base + w.tc, w.total - w.tc, st);
    if (e == LTE_ERR_UNSUPPORTED) e = launch_scores_stack(p, base + w.klin, base + w.vlin, zlin, nullptr, st);
    if (e) return e;
    return launch_ring_scatter_z(p, cache, zlin, st);
}

int lte_attn_prefill_chunk(const lte_shape* s, const lte_conv* c, void* cache, int32_t n_past, const void* q, const void* k,
                           const void* v, void* o, float* lse, void* ws, size_t ws_bytes, void* stream)
{
    return lte_attn_prefill_chunk_ex(s, c, cache, n_past, q, k, v, o, lse, 0u, ws, ws_bytes, stream);
}

int lte_attn_prefill_chunk_ex(const lte_shape* s, const lte_conv* c, void* cache, int32_t n_past, const void* q, const void* k,
                              const void* v, void* o, float* lse, uint32_t flags, void* ws, size_t ws_bytes, void* stream)
{
    int e = check_shape(s, true); if (e) return e;
    if (flags & ~LTE_CHUNK_STREAMING) return LTE_ERR_INVALID_ARG;
    const bool streaming = (flags & LTE_CHUNK_STREAMING) != 0;
    if (streaming && s->R > 4096) return LTE_ERR_UNSUPPORTED;
    e = check_conv_or_stack(s, c); if (e) return e;
    if (!cache || !q || !k || !v || !o || !lse || n_past < 0) return LTE_ERR_INVALID_ARG;
    if (!aligned16(cache) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return LTE_ERR_INVALID_ARG;
    const size_t G = s->group > 1 ? s->group : 1, bhq = (size_t)s->B * s->H * G;
    if ((double)bhq * ((double)s->R + s->W + s->T) * s->d > 2.0e10 || (double)n_past + s->T > 2.0e9) return LTE_ERR_UNSUPPORTED;
    const ChunkPlan w = chunk_plan(s, c, streaming);
    if (!ws || ((uintptr_t)ws & 255u) != 0 || ws_bytes < w.total) return LTE_ERR_WORKSPACE;
    e = check_arch(); if (e) return e;
    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)ws;
    // the local sequence: pool rows (once anything has left the window), the ring in time order, the chunk
    const int Tc = s->T, Wn = n_past < s->W ? n_past : s->W, R0 = n_past > s->W ? s->R : 0, qoff = R0 + Wn, Tloc = qoff + Tc;
    if (Tloc - s->W > (1 << 24)) return LTE_ERR_UNSUPPORTED;   // the selection's limit on candidates per head
    lte_shape sl = *s; sl.T = Tloc;
    Params p = make_params(&sl, c);                          // p.sink: positions of the whole sequence (the logit merge)
    Params psel = p; psel.sink = 0;                          // the selection sees sink tokens as +inf logits instead
    Params patt = p; patt.qoff = qoff;                       // the queries are the chunk's: positions qoff .. Tloc-1
    float* z = (float*)(base + w.z); float* zrank = (float*)(base + w.zrank); float* zsrc = (float*)(base + w.zsrc);
    int32_t* oldpos = (int32_t*)(base + w.oldpos); int32_t* idx = (int32_t*)(base + w.idx); int32_t* cnt = (int32_t*)(base + w.cnt);
    int32_t* gate = (int32_t*)(base + w.gate);
    e = launch_chunk_gather(p, cache, k, v, base + w.klin, base + w.vlin, zsrc, oldpos, gate, n_past, R0, Wn, st); if (e) return e;
    if (p.stack) {
        e = launch_scores_stack_tc(p, base + w.klin, base + w.vlin, z, nullptr, base + w.sub, w.att - w.sub, st);
        if (e == LTE_ERR_UNSUPPORTED) e = launch_scores_stack(p, base + w.klin, base + w.vlin, z, nullptr, st);
    } else {
        e = launch_scores(p, base + w.klin, base + w.vlin, z, nullptr, st);
    }
    if (e) return e;
    e = launch_chunk_merge_z(p, z, zrank, zsrc, oldpos, n_past, R0, Wn, st); if (e) return e;
    if (streaming) {
        // token by token: the pool every query sees is the streaming rule's at that query.  The entries that are in the
        // pool at some query, each with the query from which it is gone, feed the row-by-row attention kernel (the tiled
        // tensor-core kernels know prefixes of a list only); the survivors are the new pool.
        int32_t* ulist = (int32_t*)(base + w.ulist); int32_t* leave = (int32_t*)(base + w.leave); int32_t* ucnt = (int32_t*)(base + w.ucnt);
        e = launch_chunk_stream(psel, zrank, oldpos, ulist, leave, ucnt, idx, cnt, w.ucap, n_past, R0, Wn, st); if (e) return e;
        Params pu = patt; pu.R = w.ucap;                      // the entry list's row length
        // bf16: the tiled kernel with the leave times as one more mask on its retained tiles (d = 64), else row by row
        if (s->dtype == LTE_BF16) e = launch_prefill_tc(pu, q, base + w.klin, base + w.vlin, ulist, ucnt, o, lse, base + w.att, w.total - w.att, st, leave);
        else e = launch_prefill_simt(pu, q, base + w.klin, base + w.vlin, ulist, ucnt, o, lse, st, leave);
    } else {
        e = launch_select(psel, zrank, idx, cnt, nullptr, st); if (e) return e;
        // the attention kernels take the chunk's q, o, lse as they are: query row r stands at position qoff + r
        if (s->dtype == LTE_BF16) e = launch_prefill_tc(patt, q, base + w.klin, base + w.vlin, idx, cnt, o, lse, base + w.att, w.total - w.att, st);
        else e = launch_prefill_simt(patt, q, base + w.klin, base + w.vlin, idx, cnt, o, lse, st);
    }
    if (e) return e;
    return launch_chunk_commit(p, cache, base + w.klin, base + w.vlin, z, idx, cnt, oldpos, gate, n_past, n_past + Tc, R0, Wn, st);
}

int lte_attn_decode(const lte_shape* s, const lte_conv* c, void* cache, const void* q1, const void* k1,
                    const void* v1, void* o1, float* lse1, void* stream)
{
    int e = check_shape(s, false); if (e) return e;
    e = check_conv_or_stack(s, c); if (e) return e;
    if (!cache || !q1 || !k1 || !v1 || !o1 || !lse1) return LTE_ERR_INVALID_ARG;
    if (!aligned16(cache) || !aligned16(q1) || !aligned16(k1) || !aligned16(v1)) return LTE_ERR_INVALID_ARG;
    e = check_arch(); if (e) return e;
    return launch_decode(make_params(s, c), cache, q1, k1, v1, o1, lse1, (cudaStream_t)stream);
}

int lte_sparsity_stats(const lte_shape* s, const float* z, const float* lambda_or_null, float* count, float* penalty,
                       void* ws, size_t ws_bytes, void* stream)
{
    int e = check_shape(s, true); if (e) return e;
    if (!z || !count || !penalty) return LTE_ERR_INVALID_ARG;
    if (s->H > 8192) return LTE_ERR_UNSUPPORTED;
    if (!ws || ((uintptr_t)ws & 15u) != 0 || ws_bytes < (size_t)s->B * s->H * 2 * sizeof(float)) return LTE_ERR_WORKSPACE;
    e = check_arch(); if (e) return e;
    return launch_sparsity_stats(make_params(s, nullptr), z, lambda_or_null, count, penalty, (float*)ws, s->tau, (cudaStream_t)stream);
}

int lte_lambda_update(int32_t n, float* lambda, float* cbar, const float* count, int64_t step, const lte_lambda_cfg* cfg)
{
    if (n < 0 || (n > 0 && (!lambda || !cbar || !count)) || step < 0) return LTE_ERR_INVALID_ARG;
    lte_lambda_cfg d;
    d.period = 32; d.cap = 512.f; d.alpha = 1.2f; d.band = 0.95f; d.floor = 1e-9f; d.max = 1.f;
    if (cfg) d = *cfg;
    if (d.period <= 0 || !(d.alpha > 1.f) || !(d.cap > 0.f) || !(d.band > 0.f && d.band <= 1.f) || !(d.floor > 0.f) || !(d.max >= d.floor))
        return LTE_ERR_INVALID_ARG;
    const double a = 2.0 / (1.0 + d.period / 2.0);          // the new sample's weight in the moving average
    const bool adjust = step % d.period == 0;
    for (int32_t i = 0; i < n; ++i) {
        const double cb = (1.0 - a) * (double)cbar[i] + a * (double)count[i];
        cbar[i] = (float)cb;
        if (!adjust) continue;
        double l = lambda[i];
        if (cb > d.cap) l *= d.alpha;
        else if (cb < (double)d.band * d.cap) l /= d.alpha;
        if (l > d.max) l = d.max;
        if (l < d.floor) l = 0.0;
        if (cb > d.cap && l == 0.0) l = d.floor;
        lambda[i] = (float)l;
    }
    return LTE_OK;
}

int lte_attn_bwd(const lte_shape* s, const lte_conv* c, const void* q, const void* k, const void* v, const void* o,
                 const float* lse, const void* dO, const float* z, const int32_t* idx, const int32_t* cnt,
                 const float* lambda_or_null, void* dq, void* dk, void* dv, float* dw, float* dbias_or_null,
                 uint32_t flags, void* ws, size_t ws_bytes, void* stream)
{
    int e = check_shape(s, true); if (e) return e;
    if (c && c->w && c->n_layers == 3) {                   // the paper's stack: d = 64 or 32, gradients packed like the parameters
        if (c->kernel != 3 || c->dilation != 2 || (s->d != 64 && s->d != 32)) return LTE_ERR_UNSUPPORTED;
        if (s->W < 7 || !aligned16(c->w)) return LTE_ERR_INVALID_ARG;
    } else {
        e = check_conv(s, c); if (e) return e;
    }
    if (!q || !k || !v || !o || !lse || !dO || !z || !cnt || (s->R > 0 && !idx) || !dq || !dk || !dv || !dw)
        return LTE_ERR_INVALID_ARG;
    if (flags & ~LTE_BWD_CNN_INPUT_GRAD) return LTE_ERR_INVALID_ARG;
    Params p = make_params(s, c);
    if (!ws || !aligned16(ws) || ws_bytes < bwd_workspace_bytes(p, flags)) return LTE_ERR_WORKSPACE;
    e = check_arch(); if (e) return e;
    return launch_bwd(p, q, k, v, o, lse, dO, z, idx, cnt, lambda_or_null, dq, dk, dv, dw, dbias_or_null, flags, ws,
                      (cudaStream_t)stream);
}


/* ---- backward without any caller- or library-side allocation ------------------------------------------------
 * Scratch for lte_attn_bwd_static lives in this fixed array instead of a caller-supplied workspace.  Every GPU
 * that loads the library carries these LTE_STATIC_SCRATCH_BYTES until the process exits.  The symbol below is
 * only a host-side handle; the address the kernels use is resolved once per device with cudaGetSymbolAddress. */
static __device__ __align__(256) unsigned char g_bwd_static_scratch[LTE_STATIC_SCRATCH_BYTES];

namespace {
/* Device address of the scratch array on the current device (resolved on first use, per device ordinal), or NULL. */
void* static_scratch_for_current_device()
{
    static PerDevice<void*> table;
    void* p = nullptr;
    const int e = table.get(&p, [](void** out) {
        return cuda_status(cudaGetSymbolAddress(out, g_bwd_static_scratch));
    });
    return e == LTE_OK ? p : nullptr;
}
}  // namespace

/* Diagnostic for the per-device table every launcher keeps its once-per-device facts in (SM count, raised shared-memory
 * limits, symbol addresses): looks `dev` up in a table of its own and returns how many times the table has run the
 * initialiser for that device so far: 1, however many threads ask at once.  Touches no GPU. */
int lte_selftest_per_device(int dev)
{
    static PerDevice<int> table;
    static std::atomic<int> inits[kMaxDevices];
    if (dev < 0 || dev >= kMaxDevices) return LTE_ERR_INVALID_ARG;
    int v = 0;
    const int e = table.get_for(dev, &v, [dev](int* out) { *out = dev + 1000; inits[dev].fetch_add(1); return (int)LTE_OK; });
    if (e != LTE_OK || v != dev + 1000) return LTE_ERR_DEVICE_STATUS;
    return inits[dev].load();
}

int lte_attn_bwd_static(const lte_shape* s, const lte_conv* c, const void* q, const void* k, const void* v,
                        const void* o, const float* lse, const void* dO, const float* z, const int32_t* idx,
                        const int32_t* cnt, const float* lambda_or_null, void* dq, void* dk, void* dv, float* dw,
                        float* dbias_or_null, uint32_t flags, void* stream)
{
    int e = check_shape(s, true); if (e) return e;
    e = check_conv(s, c); if (e) return e;
    if (!q || !k || !v || !o || !lse || !dO || !z || !cnt || (s->R > 0 && !idx) || !dq || !dk || !dv || !dw)
        return LTE_ERR_INVALID_ARG;
    if (flags & ~LTE_BWD_CNN_INPUT_GRAD) return LTE_ERR_INVALID_ARG;
    Params p = make_params(s, c);
    if (bwd_workspace_bytes(p, flags) > (size_t)LTE_STATIC_SCRATCH_BYTES) return LTE_ERR_WORKSPACE;   /* too large for the fixed array */
    e = check_arch(); if (e) return e;
    void* scratch = static_scratch_for_current_device();
    if (!scratch) return LTE_ERR_CUDA;
    return launch_bwd(p, q, k, v, o, lse, dO, z, idx, cnt, lambda_or_null, dq, dk, dv, dw, dbias_or_null, flags,
                      scratch, (cudaStream_t)stream);
}

}  // extern "C"
