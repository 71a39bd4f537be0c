// C ABI of the compressed-KV decode path: host-side validation, cache layout,
// static work schedule, launches.  No device memory is allocated here.
#include "../../include/zsm.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <queue>
#include <unordered_map>
#include <vector>

#include "zsm_decode.cuh"
#include "zsm_decode_split.cuh"
#include "zsm_noalloc.cuh"
#include "zsm_prefill.cuh"
#include "zsm_prefill_full.cuh"

using namespace zsm;

namespace {

constexpr size_t kAlign = 256;
constexpr int kMaxSmemPerCta = 232448;  // 227 KiB opt-in limit on sm_100
constexpr int kMaxSmemPerSm = 233472;   // 228 KiB per SM, of which each resident CTA reserves 1 KiB

inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

int elem_size(int dtype) { return dtype == ZSM_F32 ? 4 : 2; }

struct Layout {
    size_t status, counters, sched_all_off, sched_all_desc;
    std::vector<size_t> sched_layer_off, sched_layer_desc;
    size_t layer_desc;  // descriptors in plain (layer, b, h) order
    size_t total;
    std::vector<UnitDesc> desc;  // [n_units], offsets filled
};

struct Shape {
    int L, B, Hq, Hkv, D, dtype, G, esz, row_bytes;
    int n_units, upl;  // units per layer
};

}  // namespace

struct zsm_cache {
    Shape s;
    float lambda, alpha, scale;
    int cosine;                       // slot similarity: 0 raw dot product, 1 cosine
    std::vector<int32_t> Bp, Bc, Br;  // [L*Hkv]
    uint8_t *base;
    size_t bytes;
    Layout lay;
    int n_sm;
    // Launch plan of the fused decode kernel, one for the all-layer launch and one for a
    // single layer's: a launch with no more units than SMs runs the wide form (one CTA per SM,
    // sixteen consumer warps, the whole shared memory as ring), otherwise two CTAs per SM.
    struct Plan {
        int ctas_per_sm, consumer_warps, stages, smem_bytes, grid;
        bool wide;
        // Split form, for a launch with at most half as many units as SMs: `split` CTAs (a
        // cluster) share each unit; 0 = not used.
        int split, split_warps, split_stages, split_smem, split_l_stride, split_kr_rows;
    } plan_all, plan_layer;
    int l_stride, br_max, br_max_pad, cap_max;
    int smem_bytes;
    std::vector<int> layer_cap_max, layer_br_max;
    // Which layer the last call enqueued on a stream wrote (kWroteAll: every layer).  A per-layer
    // decode launch may read its layer's cache before the stream's preceding kernel has finished
    // only if that kernel is known not to write it: the last call on the same stream was this
    // library's and wrote a different single layer.  (Whatever else the caller put in between
    // was launched the ordinary way, after our call had completed.)
    // Pipelined host-buffer steps (zsm_decode_step_host_async): two copy streams and three
    // events per staging half, created on first use.
    cudaStream_t cs_in = nullptr, cs_out = nullptr;
    cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_kernel[2] = {nullptr, nullptr},
                ev_out[2] = {nullptr, nullptr};
    bool slot_used[2] = {false, false};
    static constexpr int32_t kWroteAll = -1;
    std::unordered_map<cudaStream_t, int32_t> last_write;
    void wrote(cudaStream_t s, int32_t layer) {
        if (last_write.size() > 256) last_write.clear();
        last_write[s] = layer;
    }
    void wrote_everywhere() {
        for (auto &kv : last_write) kv.second = kWroteAll;
    }
    bool may_read_early(cudaStream_t s, int32_t layer) const {
        if (layer < 0) return false;
        const auto it = last_write.find(s);
        return it != last_write.end() && it->second != kWroteAll && it->second != layer;
    }
};

namespace {

bool check_config(const zsm_config_t *c) {
    if (!c) return false;
    if (c->n_layers < 1 || c->batch < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1) return false;
    if (c->n_q_heads % c->n_kv_heads != 0) return false;
    if (c->head_dim < 1) return false;
    if (c->dtype != ZSM_F32 && c->dtype != ZSM_F16 && c->dtype != ZSM_BF16) return false;
    if (!c->budget_p || !c->budget_c || !c->budget_r) return false;
    if (!(c->lambda >= 0.f && c->lambda <= 1.f)) return false;
    if (!(c->alpha >= 0.f && c->alpha <= 1.f)) return false;
    if (!(c->softmax_scale >= 0.f)) return false;
    if (c->tune_stages < 0 || c->tune_ctas_per_sm < 0 || c->tune_consumer_warps < 0) return false;
    if (c->similarity != 0 && c->similarity != 1) return false;
    if (c->tune_split != 0 && c->tune_split != 1 && c->tune_split != 2 && c->tune_split != 4 &&
        c->tune_split != 8)
        return false;
    const long n = (long)c->n_layers * c->n_kv_heads;
    for (long i = 0; i < n; ++i) {
        if (c->budget_p[i] < 0 || c->budget_c[i] < 0 || c->budget_r[i] < 0) return false;
        if ((long)c->budget_p[i] + c->budget_c[i] < 1) return false;
        if ((long)c->budget_p[i] + c->budget_c[i] + c->budget_r[i] > (1 << 24)) return false;
    }
    return true;
}

bool supported_shape(const zsm_config_t *c) {
    const int G = c->n_q_heads / c->n_kv_heads;
    if (c->head_dim != 64 && c->head_dim != 128) return false;
    if (G != 1 && G != 2 && G != 4 && G != 8) return false;
    return true;
}

Shape make_shape(const zsm_config_t *c) {
    Shape s;
    s.L = c->n_layers;
    s.B = c->batch;
    s.Hq = c->n_q_heads;
    s.Hkv = c->n_kv_heads;
    s.D = c->head_dim;
    s.dtype = c->dtype;
    s.G = s.Hq / s.Hkv;
    s.esz = elem_size(s.dtype);
    s.row_bytes = s.D * s.esz;
    s.upl = s.B * s.Hkv;
    s.n_units = s.L * s.upl;
    return s;
}

// Byte map of the caller's buffer.  grid_* are needed for the schedule tables.
void build_layout(const Shape &s, const int32_t *Bp, const int32_t *Bc, const int32_t *Br,
                  int grid_all, int grid_layer, Layout &lay) {
    size_t o = 0;
    auto take = [&](size_t bytes) {
        size_t at = o;
        o = align_up(o + bytes);
        return at;
    };
    lay.status = take(64);
    lay.counters = take((size_t)s.n_units * sizeof(UnitCounters));
    lay.sched_all_off = take((size_t)(grid_all + 1) * 4);
    lay.sched_all_desc = take((size_t)s.n_units * sizeof(UnitDesc));
    lay.sched_layer_off.resize(s.L);
    lay.sched_layer_desc.resize(s.L);
    for (int l = 0; l < s.L; ++l) {
        lay.sched_layer_off[l] = take((size_t)(grid_layer + 1) * 4);
        lay.sched_layer_desc[l] = take((size_t)s.upl * sizeof(UnitDesc));
    }
    lay.layer_desc = take((size_t)s.n_units * sizeof(UnitDesc));
    lay.desc.resize(s.n_units);
    for (int l = 0; l < s.L; ++l)
        for (int b = 0; b < s.B; ++b)
            for (int h = 0; h < s.Hkv; ++h) {
                const int u = (l * s.B + b) * s.Hkv + h;
                const int bp = Bp[l * s.Hkv + h], bc = Bc[l * s.Hkv + h], br = Br[l * s.Hkv + h];
                const size_t cap = (size_t)bp + bc, cap_pad = (cap + 3) & ~(size_t)3;
                const size_t br_pad = ((size_t)br + 3) & ~(size_t)3;
                UnitDesc &d = lay.desc[u];
                std::memset(&d, 0, sizeof(d));
                d.unit = u;
                d.Bp = bp;
                d.Bc = bc;
                d.Br = br;
                d.k_off = take(cap * s.row_bytes);
                d.v_off = take(cap * s.row_bytes);
                d.score_off = take(cap_pad * 4);
                d.pos_off = take(cap_pad * 4);
                d.kr_off = take((size_t)br * s.D * 4);
                d.vr_off = take((size_t)br * s.D * 4);
                d.w_off = take(br_pad * 4);
            }
    lay.total = o;
}

int default_grid(int n_units, int n_sm, int ctas_per_sm) {
    return std::max(1, std::min(n_units, n_sm * ctas_per_sm));
}

// Longest-processing-time-first assignment of units to CTAs: heaviest unit to the
// least loaded CTA.  Returns per-CTA unit lists flattened, with offsets.
void lpt_schedule(const std::vector<int> &units, const std::vector<UnitDesc> &desc, int row_bytes,
                  int D, int grid, std::vector<int32_t> &off, std::vector<int> &order) {
    auto weight = [&](int u) -> double {
        const UnitDesc &d = desc[u];
        return (double)(d.Bp + d.Bc) * (2.0 * row_bytes + 12.0) + (double)d.Br * D * 8.0 + 8192.0;
    };
    std::vector<int> sorted(units);
    std::stable_sort(sorted.begin(), sorted.end(),
                     [&](int a, int b) { return weight(a) > weight(b); });
    typedef std::pair<double, int> Load;  // (load, cta); smallest load first, then lowest cta
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> pq;
    for (int c = 0; c < grid; ++c) pq.push(Load(0.0, c));
    std::vector<std::vector<int>> per(grid);
    for (int u : sorted) {
        Load l = pq.top();
        pq.pop();
        per[l.second].push_back(u);
        pq.push(Load(l.first + weight(u), l.second));
    }
    off.assign(grid + 1, 0);
    order.clear();
    for (int c = 0; c < grid; ++c) {
        off[c] = (int32_t)order.size();
        order.insert(order.end(), per[c].begin(), per[c].end());
    }
    off[grid] = (int32_t)order.size();
}

zsm_status_t cuda_status(cudaError_t e) { return e == cudaSuccess ? ZSM_OK : ZSM_ERR_CUDA; }

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

float half_bits_to_float(uint16_t h, int dtype) {
    if (dtype == ZSM_F16) {
        __half_raw r;
        r.x = h;
        return __half2float(__half(r));
    }
    uint32_t u = (uint32_t)h << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

uint16_t float_to_half_bits(float f, int dtype) {
    if (dtype == ZSM_F16) {
        __half_raw r = static_cast<__half_raw>(__float2half_rn(f));
        return r.x;
    }
    __nv_bfloat16_raw r = static_cast<__nv_bfloat16_raw>(__float2bfloat16_rn(f));
    return r.x;
}

// Shared-memory plan of the decode kernel for (stages, warps); returns total bytes.
int decode_smem_total(const zsm_cache *c, int stages, int warps) {
    return (int)decode_smem_layout(stages, c->s.G, c->s.D, c->s.row_bytes, c->l_stride,
                                   c->br_max_pad, warps)
        .total;
}

}  // namespace

extern "C" {

const char *zsm_status_string(zsm_status_t s) {
    switch (s) {
        case ZSM_OK: return "ok";
        case ZSM_ERR_INVALID_ARG: return "invalid argument";
        case ZSM_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case ZSM_ERR_STATE: return "call not valid in this state";
        case ZSM_ERR_CUDA: return "CUDA runtime error";
        case ZSM_ERR_UNSUPPORTED: return "unsupported shape";
        case ZSM_ERR_DEVICE_CHECK: return "device-side check failed";
        case ZSM_ERR_TIMEOUT: return "device-side wait timed out";
        case ZSM_ERR_NO_MEMORY: return "out of host memory";
    }
    return "unknown status";
}

zsm_status_t zsm_split_budget(int32_t B, float tail_ratio, float dense_ratio, int32_t *Bp,
                              int32_t *Bc, int32_t *Br) {
    if (!Bp || !Bc || !Br || B < 1) return ZSM_ERR_INVALID_ARG;
    if (!(tail_ratio >= 0.f && tail_ratio <= 1.f) || !(dense_ratio >= 0.f && dense_ratio <= 1.f))
        return ZSM_ERR_INVALID_ARG;
    const double tr = (double)tail_ratio, dr = (double)dense_ratio;
    // ratios arrive as floats; snap them to the decimal the caller most likely wrote
    const double trs = std::round(tr * 1e6) / 1e6, drs = std::round(dr * 1e6) / 1e6;
    int32_t bp = (int32_t)std::floor(trs * (double)B);
    int32_t rest = B - bp, br = 0;
    if (drs > 0.0 && rest > 0) {
        br = (int32_t)std::floor(drs * (double)rest + 0.5);
        br = std::max(br, 1);
        br = std::min(br, rest);
    }
    int32_t bc = rest - br;
    if (bp + bc < 1 && br > 0) {
        br -= 1;
        bc += 1;
    }
    *Bp = bp;
    *Bc = bc;
    *Br = br;
    return ZSM_OK;
}

zsm_status_t zsm_cache_bytes(const zsm_config_t *cfg, size_t *bytes) {
    if (!bytes || !check_config(cfg)) return ZSM_ERR_INVALID_ARG;
    const Shape s = make_shape(cfg);
    Layout lay;
    // schedule tables are sized for the largest grid any device of this family can ask for
    const int grid_cap_all = std::min(s.n_units, 1024);
    const int grid_cap_layer = std::min(s.upl, 1024);
    build_layout(s, cfg->budget_p, cfg->budget_c, cfg->budget_r, grid_cap_all, grid_cap_layer, lay);
    *bytes = lay.total;
    return ZSM_OK;
}

zsm_status_t zsm_cache_create(const zsm_config_t *cfg, void *dev_buf, size_t bytes,
                              zsm_cache_t **out) {
    if (!out) return ZSM_ERR_INVALID_ARG;
    *out = nullptr;
    if (!check_config(cfg) || !dev_buf) return ZSM_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(dev_buf) % kAlign != 0) return ZSM_ERR_INVALID_ARG;
    if (!supported_shape(cfg)) return ZSM_ERR_UNSUPPORTED;
    size_t need = 0;
    zsm_status_t st = zsm_cache_bytes(cfg, &need);
    if (st != ZSM_OK) return st;
    if (bytes < need) return ZSM_ERR_BUFFER_TOO_SMALL;

    zsm_cache *c = new (std::nothrow) zsm_cache();
    if (!c) return ZSM_ERR_NO_MEMORY;
    c->s = make_shape(cfg);
    const Shape &s = c->s;
    c->lambda = cfg->lambda;
    c->alpha = cfg->alpha;
    c->cosine = cfg->similarity;
    c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt((float)s.D);
    const int nh = s.L * s.Hkv;
    c->Bp.assign(cfg->budget_p, cfg->budget_p + nh);
    c->Bc.assign(cfg->budget_c, cfg->budget_c + nh);
    c->Br.assign(cfg->budget_r, cfg->budget_r + nh);
    c->base = static_cast<uint8_t *>(dev_buf);
    c->bytes = bytes;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&c->n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        delete c;
        return ZSM_ERR_CUDA;
    }

    c->cap_max = 0;
    c->br_max = 0;
    int ent_max = 0;
    c->layer_cap_max.assign(s.L, 0);
    c->layer_br_max.assign(s.L, 0);
    for (int i = 0; i < nh; ++i) {
        const int cap = c->Bp[i] + c->Bc[i];
        c->cap_max = std::max(c->cap_max, cap);
        c->br_max = std::max(c->br_max, c->Br[i]);
        ent_max = std::max(ent_max, cap + c->Br[i] + 1);
        c->layer_cap_max[i / s.Hkv] = std::max(c->layer_cap_max[i / s.Hkv], cap);
        c->layer_br_max[i / s.Hkv] = std::max(c->layer_br_max[i / s.Hkv], c->Br[i]);
    }
    c->br_max_pad = (c->br_max + 3) & ~3;
    c->l_stride = (ent_max + 3) & ~3;

    // ---- launch plans of the fused decode kernel ----
    if (c->br_max > prefill_max_residual(s.D)) {
        delete c;
        return ZSM_ERR_UNSUPPORTED;
    }
    if (prepare_prefill(s.dtype, s.D) != 0 ||
        (s.dtype != ZSM_F32 && prepare_full_scores(s.dtype, s.D) != 0)) {
        delete c;
        return ZSM_ERR_CUDA;
    }
    const int header_bytes =
        16 + (int)sizeof(UnitDesc) + (s.G + 2) * s.row_bytes + c->br_max_pad * 4;
    if (header_bytes > kTileBytes) {
        delete c;
        return ZSM_ERR_UNSUPPORTED;
    }
    auto make_plan = [&](int units, zsm_cache::Plan &pl) -> zsm_status_t {
        const bool solo = units <= c->n_sm;  // a CTA has an SM to itself whatever we do
        pl.ctas_per_sm = cfg->tune_ctas_per_sm > 0 ? cfg->tune_ctas_per_sm : (solo ? 1 : 2);
        pl.consumer_warps = cfg->tune_consumer_warps > 0
                                ? cfg->tune_consumer_warps
                                : (pl.ctas_per_sm == 1 ? kMaxConsumerWarps : kPairConsumerWarps);
        pl.wide = pl.ctas_per_sm == 1;
        if (pl.ctas_per_sm > 8 || pl.consumer_warps > (pl.wide ? kMaxConsumerWarps : kPairConsumerWarps))
            return ZSM_ERR_INVALID_ARG;
        const int budget = kMaxSmemPerCta / pl.ctas_per_sm - 1024 * (pl.ctas_per_sm > 1);
        const int fixed = decode_smem_total(c, 0, pl.consumer_warps);
        int stages = (budget - fixed - 64) / (kTileBytes + 16);
        if (cfg->tune_stages > 0) stages = std::min(stages, (int)cfg->tune_stages);
        stages = std::min(stages, 12);
        while (stages >= 2 && decode_smem_total(c, stages, pl.consumer_warps) > budget) --stages;
        // Two CTAs per SM: a sixth stage that takes the pair past 216 KB of the SM's 228 KB buys
        // nothing and leaves the L1 almost no room (c4 at 5 %: 0.2311 ms per step against 0.2290
        // with five stages; c3, whose six stages stay below that, is 0.5 % faster with them).
        if (pl.ctas_per_sm == 2 && cfg->tune_stages == 0 && stages > 5 &&
            decode_smem_total(c, stages, pl.consumer_warps) > 108 * 1024)
            stages = 5;
        if (stages < 2) return ZSM_ERR_UNSUPPORTED;  // budget too large for the weight array
        pl.stages = stages;
        pl.smem_bytes = decode_smem_total(c, stages, pl.consumer_warps);
        int occ = 0;
        const int rc = prepare_decode_fused(s.dtype, s.D, s.G, pl.smem_bytes,
                                            (pl.consumer_warps + kExtraWarps) * 32, &occ);
        if (rc != 0) return rc == -1 ? ZSM_ERR_UNSUPPORTED : ZSM_ERR_CUDA;
        if (!pl.wide) {
            if (occ < 1) return ZSM_ERR_UNSUPPORTED;
            pl.ctas_per_sm = std::min(pl.ctas_per_sm, occ);
        }
        pl.grid = std::min(default_grid(units, c->n_sm, pl.ctas_per_sm), 1024);

        // Split form: only when nothing asks for the paired form and the launch is small.
        pl.split = 0;
        if (cfg->tune_split != 1 && cfg->tune_ctas_per_sm == 0 && units * 2 <= c->n_sm) {
            const int limit = cfg->tune_split > 1 ? cfg->tune_split : kSplitMaxCluster;
            // eight consumer warps: a launch of this form is bound by latencies, not by what its
            // warps can consume, and the smaller CTA starts sooner (c4 16.9 -> 16.4 us per layer)
            const int warps = cfg->tune_consumer_warps > 0
                                  ? std::min((int)cfg->tune_consumer_warps, kMaxConsumerWarps)
                                  : kPairConsumerWarps;
            for (int C = kSplitMaxCluster; C >= 2 && pl.split == 0; C >>= 1) {
                if (C > limit || units * C > c->n_sm) continue;
                const int ls = split_l_stride(c->cap_max, c->br_max, s.esz, C);
                // merged keys stay in shared memory on rank 0 when they are few (Eq. (hatr)) and
                // the CTA has the SM's shared memory to itself
                int kr_rows = c->br_max * s.D * 4 <= 32768 ? c->br_max : 0;
                auto total = [&](int st) {
                    return (int)split_smem_layout(st, s.G, s.D, s.row_bytes, ls, c->br_max_pad,
                                                  kr_rows, warps, C).total;
                };
                auto fit_stages = [&](int budget) {
                    int n = (budget - total(0) - 64) / (kTileBytes + 16);
                    n = std::min(n, 12);
                    while (n >= 2 && total(n) > budget) --n;
                    return n;
                };
                // Two CTAs of this shape fit on an SM when each stays within half of its shared
                // memory (less the per-CTA reserve): the next layer's launch can then settle in
                // beside this one's and have its first tiles in flight before this one ends.
                // Taken when it leaves at least five ring stages (c5's grouped heads leave three:
                // 25.5 us per layer against 23.9 with the whole SM); otherwise the whole SM.
                // (Keeping the merged keys out of shared memory to gain a stage loses: the tail
                // warp's reads of them are then the last thing the launch waits for; c4 14.9 ->
                // 16.4 us per layer.)
                const int pair_budget = kMaxSmemPerSm / 2 - 1024 - 256;
                int st = 0;
                if (warps <= kPairConsumerWarps && (cfg->tune_stages == 0 || cfg->tune_stages <= 7)) {
                    st = fit_stages(pair_budget);
                    if (cfg->tune_stages > 0) st = std::min(st, (int)cfg->tune_stages);
                    if (st < 5) st = 0;
                }
                if (st == 0) {
                    st = fit_stages(kMaxSmemPerCta);
                    if (cfg->tune_stages > 0) st = std::min(st, (int)cfg->tune_stages);
                }
                if (st < 2) continue;
                int fit = 0;
                const int rc = prepare_decode_split(s.dtype, s.D, s.G, C, total(st),
                                                    (warps + kExtraWarps) * 32, &fit);
                if (rc != 0 || fit < 1) continue;
                pl.split = C;
                pl.split_warps = warps;
                pl.split_stages = st;
                pl.split_smem = total(st);
                pl.split_l_stride = ls;
                pl.split_kr_rows = kr_rows;
            }
        }
        return ZSM_OK;
    };
    {
        zsm_status_t ps = make_plan(s.n_units, c->plan_all);
        if (ps == ZSM_OK) ps = make_plan(s.upl, c->plan_layer);
        if (ps != ZSM_OK) {
            delete c;
            return ps;
        }
    }

    // same table sizes as zsm_cache_bytes, so the byte count never depends on the device
    build_layout(s, c->Bp.data(), c->Bc.data(), c->Br.data(), std::min(s.n_units, 1024),
                 std::min(s.upl, 1024), c->lay);
    const Layout &lay = c->lay;

    // ---- tables to the device ----
    std::vector<uint8_t> host(lay.desc.empty() ? 0 : (size_t)(lay.desc[0].k_off), 0);
    auto put = [&](size_t at, const void *src, size_t n) { std::memcpy(host.data() + at, src, n); };
    std::vector<int32_t> off;
    std::vector<int> order, units;
    std::vector<UnitDesc> dl;
    units.resize(s.n_units);
    for (int u = 0; u < s.n_units; ++u) units[u] = u;
    lpt_schedule(units, lay.desc, s.row_bytes, s.D, c->plan_all.grid, off, order);
    dl.resize(order.size());
    for (size_t i = 0; i < order.size(); ++i) dl[i] = lay.desc[order[i]];
    put(lay.sched_all_off, off.data(), off.size() * 4);
    put(lay.sched_all_desc, dl.data(), dl.size() * sizeof(UnitDesc));
    for (int l = 0; l < s.L; ++l) {
        units.resize(s.upl);
        for (int u = 0; u < s.upl; ++u) units[u] = l * s.upl + u;
        lpt_schedule(units, lay.desc, s.row_bytes, s.D, c->plan_layer.grid, off, order);
        dl.resize(order.size());
        for (size_t i = 0; i < order.size(); ++i) dl[i] = lay.desc[order[i]];
        put(lay.sched_layer_off[l], off.data(), off.size() * 4);
        put(lay.sched_layer_desc[l], dl.data(), dl.size() * sizeof(UnitDesc));
    }
    put(lay.layer_desc, lay.desc.data(), lay.desc.size() * sizeof(UnitDesc));
    // status and counters are zero in `host` already
    cudaError_t e = cudaMemcpy(c->base, host.data(), host.size(), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        delete c;
        return ZSM_ERR_CUDA;
    }
    // Set-up of zsm_prefill_compress_static for this device, here because this call blocks and
    // may allocate anyway.  A failure is not this call's: the static entry point retries and
    // reports it.
    (void)static_scratch_setup();
    (void)cudaGetLastError();
    *out = c;
    return ZSM_OK;
}

zsm_status_t zsm_cache_reset(zsm_cache_t *c, zsm_stream_t stream) {
    if (!c) return ZSM_ERR_INVALID_ARG;
    c->wrote(static_cast<cudaStream_t>(stream), zsm_cache::kWroteAll);
    return cuda_status(cudaMemsetAsync(c->base + c->lay.counters, 0,
                                       (size_t)c->s.n_units * sizeof(UnitCounters),
                                       static_cast<cudaStream_t>(stream)));
}

zsm_status_t zsm_cache_free(zsm_cache_t *c) {
    if (!c) return ZSM_ERR_INVALID_ARG;
    for (int s = 0; s < 2; ++s) {
        if (c->ev_in[s]) cudaEventDestroy(c->ev_in[s]);
        if (c->ev_kernel[s]) cudaEventDestroy(c->ev_kernel[s]);
        if (c->ev_out[s]) cudaEventDestroy(c->ev_out[s]);
    }
    if (c->cs_in) cudaStreamDestroy(c->cs_in);
    if (c->cs_out) cudaStreamDestroy(c->cs_out);
    delete c;
    return ZSM_OK;
}

zsm_status_t zsm_unit_capacity(const zsm_cache_t *c, int32_t layer, int32_t h,
                               int32_t *n_token_slots, int32_t *n_residual_slots) {
    if (!c || layer < 0 || layer >= c->s.L || h < 0 || h >= c->s.Hkv) return ZSM_ERR_INVALID_ARG;
    const int i = layer * c->s.Hkv + h;
    if (n_token_slots) *n_token_slots = c->Bp[i] + c->Bc[i];
    if (n_residual_slots) *n_residual_slots = c->Br[i];
    return ZSM_OK;
}

zsm_status_t zsm_decode_launch_info(const zsm_cache_t *c, int32_t layer, int32_t *grid,
                                    int32_t *block, int32_t *dynamic_smem_bytes) {
    if (!c || layer < -1 || layer >= c->s.L) return ZSM_ERR_INVALID_ARG;
    const zsm_cache::Plan &pl = layer < 0 ? c->plan_all : c->plan_layer;
    if (pl.split >= 2) {
        if (grid) *grid = (layer < 0 ? c->s.n_units : c->s.upl) * pl.split;
        if (block) *block = (pl.split_warps + kExtraWarps) * 32;
        if (dynamic_smem_bytes) *dynamic_smem_bytes = pl.split_smem;
        return ZSM_OK;
    }
    if (grid) *grid = pl.grid;
    if (block) *block = (pl.consumer_warps + kExtraWarps) * 32;
    if (dynamic_smem_bytes) *dynamic_smem_bytes = pl.smem_bytes;
    return ZSM_OK;
}

zsm_status_t zsm_decode_step(zsm_cache_t *c, int32_t layer, const void *q, const void *k_new,
                             const void *v_new, void *out, int32_t *victim_pos,
                             int32_t *merge_slot, zsm_stream_t stream) {
    if (!c || !q || !k_new || !v_new || !out) return ZSM_ERR_INVALID_ARG;
    if (layer < -1 || layer >= c->s.L) return ZSM_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out))
        return ZSM_ERR_INVALID_ARG;
    const Layout &lay = c->lay;
    DecodeParams p;
    p.base = c->base;
    if (layer < 0) {
        p.sched_off = reinterpret_cast<const int32_t *>(c->base + lay.sched_all_off);
        p.sched_desc = reinterpret_cast<const UnitDesc *>(c->base + lay.sched_all_desc);
        p.unit_base = 0;
    } else {
        p.sched_off = reinterpret_cast<const int32_t *>(c->base + lay.sched_layer_off[layer]);
        p.sched_desc = reinterpret_cast<const UnitDesc *>(c->base + lay.sched_layer_desc[layer]);
        p.unit_base = layer * c->s.upl;
    }
    p.counters = reinterpret_cast<UnitCounters *>(c->base + lay.counters);
    p.status = reinterpret_cast<int32_t *>(c->base + lay.status);
    p.q = q;
    p.k_new = k_new;
    p.v_new = v_new;
    p.out = out;
    p.victim_pos = victim_pos;
    p.merge_slot = merge_slot;
    const zsm_cache::Plan &pl = layer < 0 ? c->plan_all : c->plan_layer;
    p.stages = pl.stages;
    p.l_stride = c->l_stride;
    p.br_max_pad = c->br_max_pad;
    p.cosine = c->cosine;
    p.lambda = c->lambda;
    p.alpha = c->alpha;
    p.scale = c->scale;
    if (pl.split >= 2) {
        SplitParams sp;
        sp.d = p;
        sp.d.sched_off = nullptr;
        sp.d.sched_desc = reinterpret_cast<const UnitDesc *>(c->base + lay.layer_desc) +
                          (layer < 0 ? 0 : (size_t)layer * c->s.upl);
        sp.d.stages = pl.split_stages;
        sp.d.l_stride = pl.split_l_stride;
        sp.n_units = layer < 0 ? c->s.n_units : c->s.upl;
        sp.kr_rows = pl.split_kr_rows;
        sp.early = c->may_read_early(static_cast<cudaStream_t>(stream), layer) ? 1 : 0;
        c->wrote(static_cast<cudaStream_t>(stream), layer < 0 ? zsm_cache::kWroteAll : layer);
        const int rs = launch_decode_split(c->s.dtype, c->s.D, c->s.G, sp, pl.split, pl.split_warps,
                                           static_cast<cudaStream_t>(stream));
        if (rs == -1) return ZSM_ERR_UNSUPPORTED;
        return rs == 0 ? ZSM_OK : ZSM_ERR_CUDA;
    }
    c->wrote(static_cast<cudaStream_t>(stream), layer < 0 ? zsm_cache::kWroteAll : layer);
    const int rc = launch_decode_fused(c->s.dtype, c->s.D, c->s.G, p, pl.grid, pl.consumer_warps,
                                       pl.wide, static_cast<cudaStream_t>(stream));
    if (rc == -1) return ZSM_ERR_UNSUPPORTED;
    return rc == 0 ? ZSM_OK : ZSM_ERR_CUDA;
}

zsm_status_t zsm_decode_staging_bytes(const zsm_cache_t *c, int32_t layer, size_t *bytes) {
    if (!c || !bytes || layer < -1 || layer >= c->s.L) return ZSM_ERR_INVALID_ARG;
    const size_t nu = layer < 0 ? c->s.n_units : c->s.upl;
    const size_t qb = align_up(nu * c->s.G * c->s.row_bytes), kb = align_up(nu * c->s.row_bytes);
    *bytes = 2 * qb + 2 * kb;
    return ZSM_OK;
}

zsm_status_t zsm_decode_step_host(zsm_cache_t *c, int32_t layer, const void *q_host,
                                  const void *k_new_host, const void *v_new_host,
                                  void *out_host, void *staging, size_t staging_bytes,
                                  zsm_stream_t stream) {
    if (!c || !q_host || !k_new_host || !v_new_host || !out_host || !staging)
        return ZSM_ERR_INVALID_ARG;
    size_t need = 0;
    zsm_status_t st = zsm_decode_staging_bytes(c, layer, &need);
    if (st != ZSM_OK) return st;
    if (staging_bytes < need) return ZSM_ERR_BUFFER_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(staging) % kAlign != 0) return ZSM_ERR_INVALID_ARG;
    const size_t nu = layer < 0 ? c->s.n_units : c->s.upl;
    const size_t qn = nu * c->s.G * c->s.row_bytes, kn = nu * c->s.row_bytes;
    const size_t qb = align_up(qn), kb = align_up(kn);
    uint8_t *sq = static_cast<uint8_t *>(staging), *sk = sq + qb, *sv = sk + kb, *so = sv + kb;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(sq, q_host, qn, cudaMemcpyHostToDevice, cs);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sk, k_new_host, kn, cudaMemcpyHostToDevice, cs);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sv, v_new_host, kn, cudaMemcpyHostToDevice, cs);
    if (e != cudaSuccess) return ZSM_ERR_CUDA;
    st = zsm_decode_step(c, layer, sq, sk, sv, so, nullptr, nullptr, stream);
    if (st != ZSM_OK) return st;
    e = cudaMemcpyAsync(out_host, so, qn, cudaMemcpyDeviceToHost, cs);
    if (e == cudaSuccess) e = cudaStreamSynchronize(cs);
    return cuda_status(e);
}

zsm_status_t zsm_decode_host_layout(const zsm_cache_t *c, int32_t layer, size_t *q_off,
                                    size_t *k_off, size_t *v_off, size_t *in_bytes,
                                    size_t *out_bytes) {
    if (!c || layer < -1 || layer >= c->s.L) return ZSM_ERR_INVALID_ARG;
    const size_t nu = layer < 0 ? c->s.n_units : c->s.upl;
    const size_t qb = align_up(nu * c->s.G * c->s.row_bytes), kb = align_up(nu * c->s.row_bytes);
    if (q_off) *q_off = 0;
    if (k_off) *k_off = qb;
    if (v_off) *v_off = qb + kb;
    if (in_bytes) *in_bytes = qb + 2 * kb;
    if (out_bytes) *out_bytes = nu * c->s.G * c->s.row_bytes;
    return ZSM_OK;
}

zsm_status_t zsm_decode_step_host_async(zsm_cache_t *c, int32_t layer, const void *in_host,
                                        void *out_host, void *staging, size_t staging_bytes,
                                        int32_t slot, zsm_stream_t stream) {
    if (!c || !in_host || !out_host || !staging || (slot != 0 && slot != 1))
        return ZSM_ERR_INVALID_ARG;
    size_t k_off = 0, v_off = 0, in_bytes = 0, out_bytes = 0;
    zsm_status_t st = zsm_decode_host_layout(c, layer, nullptr, &k_off, &v_off, &in_bytes, &out_bytes);
    if (st != ZSM_OK) return st;
    const size_t half = in_bytes + align_up(out_bytes);
    if (staging_bytes < 2 * half) return ZSM_ERR_BUFFER_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(staging) % kAlign != 0) return ZSM_ERR_INVALID_ARG;
    if (!c->cs_in) {
        bool ok = cudaStreamCreateWithFlags(&c->cs_in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&c->cs_out, cudaStreamNonBlocking) == cudaSuccess;
        for (int s = 0; s < 2 && ok; ++s)
            ok = cudaEventCreateWithFlags(&c->ev_in[s], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&c->ev_kernel[s], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&c->ev_out[s], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return ZSM_ERR_CUDA;
    }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    uint8_t *sin = static_cast<uint8_t *>(staging) + (size_t)slot * half, *sout = sin + in_bytes;
    cudaError_t e = cudaSuccess;
    // copy in, once the kernel that last read this half has finished
    if (c->slot_used[slot]) e = cudaStreamWaitEvent(c->cs_in, c->ev_kernel[slot], 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sin, in_host, in_bytes, cudaMemcpyHostToDevice, c->cs_in);
    if (e == cudaSuccess) e = cudaEventRecord(c->ev_in[slot], c->cs_in);
    // the step, once its inputs are in and the previous result of this half has left
    if (e == cudaSuccess) e = cudaStreamWaitEvent(cs, c->ev_in[slot], 0);
    if (e == cudaSuccess && c->slot_used[slot]) e = cudaStreamWaitEvent(cs, c->ev_out[slot], 0);
    if (e != cudaSuccess) return ZSM_ERR_CUDA;
    st = zsm_decode_step(c, layer, sin, sin + k_off, sin + v_off, sout, nullptr, nullptr, stream);
    if (st != ZSM_OK) return st;
    e = cudaEventRecord(c->ev_kernel[slot], cs);
    // copy out
    if (e == cudaSuccess) e = cudaStreamWaitEvent(c->cs_out, c->ev_kernel[slot], 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_host, sout, out_bytes, cudaMemcpyDeviceToHost, c->cs_out);
    if (e == cudaSuccess) e = cudaEventRecord(c->ev_out[slot], c->cs_out);
    c->slot_used[slot] = true;
    return cuda_status(e);
}

zsm_status_t zsm_decode_step_host_wait(zsm_cache_t *c, int32_t slot) {
    if (!c || (slot != 0 && slot != 1)) return ZSM_ERR_INVALID_ARG;
    if (!c->slot_used[slot]) return ZSM_ERR_STATE;
    return cuda_status(cudaEventSynchronize(c->ev_out[slot]));
}

zsm_status_t zsm_prefill_workspace_bytes(const zsm_cache_t *c, int32_t T, int32_t W,
                                         size_t *bytes) {
    if (!c || !bytes || T < 1 || W < 0 || W > T) return ZSM_ERR_INVALID_ARG;
    *bytes = prefill_workspace_layout(c->s.upl, T, c->s.G * W).total;
    return ZSM_OK;
}

zsm_status_t zsm_prefill_compress(zsm_cache_t *c, int32_t layer, const void *K, const void *V,
                                  const void *Qw, const float *scores, int32_t T, int32_t W,
                                  void *workspace, size_t workspace_bytes, float *dbg_scores,
                                  uint8_t *dbg_evicted, int32_t *dbg_targets,
                                  zsm_stream_t stream) {
    if (!c || !K || !V || !workspace) return ZSM_ERR_INVALID_ARG;
    if (layer < 0 || layer >= c->s.L || T < 1) return ZSM_ERR_INVALID_ARG;
    if (!Qw && !scores) return ZSM_ERR_INVALID_ARG;
    if (Qw && (W < 1 || W > T)) return ZSM_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(V) || (Qw && !aligned16(Qw))) return ZSM_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % kAlign != 0) return ZSM_ERR_INVALID_ARG;
    const int w_eff = Qw ? W : 0;
    PrefillParams p;
    p.wl = prefill_workspace_layout(c->s.upl, T, c->s.G * w_eff);
    if (workspace_bytes < p.wl.total) return ZSM_ERR_BUFFER_TOO_SMALL;
    p.base = c->base;
    p.desc = reinterpret_cast<const UnitDesc *>(c->base + c->lay.layer_desc) + (size_t)layer * c->s.upl;
    p.counters = reinterpret_cast<UnitCounters *>(c->base + c->lay.counters);
    p.status = reinterpret_cast<int32_t *>(c->base + c->lay.status);
    p.K = K;
    p.V = V;
    p.Qw = Qw;
    p.scores_in = Qw ? nullptr : scores;
    p.ws = static_cast<uint8_t *>(workspace);
    p.dbg_scores = dbg_scores;
    p.dbg_evicted = dbg_evicted;
    p.dbg_targets = dbg_targets;
    p.units = c->s.upl;
    p.T = T;
    p.W = w_eff;
    p.G = c->s.G;
    p.n_kv_heads = c->s.Hkv;
    p.n_sm = c->n_sm;
    p.max_cap = c->layer_cap_max[layer];
    p.cosine = c->cosine;
    p.lambda = c->lambda;
    p.scale = c->scale;
    c->wrote(static_cast<cudaStream_t>(stream), layer);
    const int rc = launch_prefill(c->s.dtype, c->s.D, p, std::max(1, c->layer_br_max[layer]),
                                  static_cast<cudaStream_t>(stream));
    if (rc == -1) return ZSM_ERR_UNSUPPORTED;
    return rc == 0 ? ZSM_OK : ZSM_ERR_CUDA;
}

zsm_status_t zsm_prefill_scores_full_workspace_bytes(const zsm_cache_t *c, int32_t T,
                                                     size_t *bytes) {
    if (!c || !bytes || T < 1) return ZSM_ERR_INVALID_ARG;
    *bytes = align_up((size_t)c->s.B * c->s.Hq * T * sizeof(float));
    return ZSM_OK;
}

zsm_status_t zsm_prefill_scores_full(zsm_cache_t *c, const void *K, const void *Q,
                                     const float *lse, int32_t T, float *scores,
                                     void *workspace, size_t workspace_bytes,
                                     zsm_stream_t stream) {
    if (!c || !K || !Q || !scores || T < 1) return ZSM_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(Q)) return ZSM_ERR_INVALID_ARG;
    if (c->s.dtype == ZSM_F32) return ZSM_ERR_UNSUPPORTED;
    if (!lse) {
        size_t need = 0;
        zsm_prefill_scores_full_workspace_bytes(c, T, &need);
        if (!workspace || reinterpret_cast<uintptr_t>(workspace) % kAlign != 0)
            return ZSM_ERR_INVALID_ARG;
        if (workspace_bytes < need) return ZSM_ERR_BUFFER_TOO_SMALL;
    }
    if ((long)c->s.B * c->s.Hq > 65535) return ZSM_ERR_UNSUPPORTED;
    FullScoreParams p;
    p.K = K;
    p.Q = Q;
    p.lse = lse;
    p.lse_out = lse ? nullptr : static_cast<float *>(workspace);
    p.scores = scores;
    p.status = reinterpret_cast<int32_t *>(c->base + c->lay.status);
    p.batch = c->s.B;
    p.n_kv_heads = c->s.Hkv;
    p.G = c->s.G;
    p.T = T;
    p.lambda = c->lambda;
    p.scale = c->scale;
    const int rc = launch_full_scores(c->s.dtype, c->s.D, p, static_cast<cudaStream_t>(stream));
    if (rc == -1) return ZSM_ERR_UNSUPPORTED;
    return rc == 0 ? ZSM_OK : ZSM_ERR_CUDA;
}

zsm_status_t zsm_prefill_attention(zsm_cache_t *c, const void *K, const void *V, const void *Q,
                                   int32_t T, void *out, float *lse, float *scores,
                                   zsm_stream_t stream) {
    if (!c || !K || !V || !Q || !out || !lse || T < 1) return ZSM_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(V) || !aligned16(Q) || !aligned16(out)) return ZSM_ERR_INVALID_ARG;
    if (c->s.dtype == ZSM_F32) return ZSM_ERR_UNSUPPORTED;
    if ((long)c->s.B * c->s.Hq > 65535) return ZSM_ERR_UNSUPPORTED;
    FullScoreParams p;
    p.K = K;
    p.Q = Q;
    p.status = reinterpret_cast<int32_t *>(c->base + c->lay.status);
    p.batch = c->s.B;
    p.n_kv_heads = c->s.Hkv;
    p.G = c->s.G;
    p.T = T;
    p.lambda = c->lambda;
    p.scale = c->scale;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    // one pass gives the output and the rows' log-sum-exp ...
    p.lse = nullptr;
    p.lse_out = lse;
    p.scores = nullptr;
    int rc = launch_attention_output(c->s.dtype, c->s.D, p, V, out, cs);
    if (rc == -1) return ZSM_ERR_UNSUPPORTED;
    if (rc != 0) return ZSM_ERR_CUDA;
    if (!scores) return ZSM_OK;
    // ... from which the decayed column sums follow
    p.lse = lse;
    p.lse_out = nullptr;
    p.scores = scores;
    rc = launch_full_scores(c->s.dtype, c->s.D, p, cs);
    if (rc == -1) return ZSM_ERR_UNSUPPORTED;
    return rc == 0 ? ZSM_OK : ZSM_ERR_CUDA;
}

zsm_status_t zsm_cache_export_unit(zsm_cache_t *c, int32_t layer, int32_t b, int32_t h,
                                   float *K, float *V, float *score, int32_t *pos, float *Kr,
                                   float *Vr, uint32_t *w, int32_t *counters,
                                   zsm_stream_t stream) {
    if (!c || layer < 0 || layer >= c->s.L || b < 0 || b >= c->s.B || h < 0 || h >= c->s.Hkv)
        return ZSM_ERR_INVALID_ARG;
    const Shape &s = c->s;
    const UnitDesc &d = c->lay.desc[(layer * s.B + b) * s.Hkv + h];
    const size_t cap = (size_t)d.Bp + d.Bc;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(cs) != cudaSuccess) return ZSM_ERR_CUDA;
    std::vector<uint8_t> raw(cap * s.row_bytes);
    for (int which = 0; which < 2; ++which) {
        float *dst = which ? V : K;
        if (!dst) continue;
        if (cudaMemcpy(raw.data(), c->base + (which ? d.v_off : d.k_off), raw.size(),
                       cudaMemcpyDeviceToHost) != cudaSuccess)
            return ZSM_ERR_CUDA;
        if (s.dtype == ZSM_F32) {
            std::memcpy(dst, raw.data(), raw.size());
        } else {
            const uint16_t *hsrc = reinterpret_cast<const uint16_t *>(raw.data());
            for (size_t i = 0; i < cap * s.D; ++i) dst[i] = half_bits_to_float(hsrc[i], s.dtype);
        }
    }
    cudaError_t e = cudaSuccess;
    if (score && e == cudaSuccess)
        e = cudaMemcpy(score, c->base + d.score_off, cap * 4, cudaMemcpyDeviceToHost);
    if (pos && e == cudaSuccess)
        e = cudaMemcpy(pos, c->base + d.pos_off, cap * 4, cudaMemcpyDeviceToHost);
    if (Kr && d.Br > 0 && e == cudaSuccess)
        e = cudaMemcpy(Kr, c->base + d.kr_off, (size_t)d.Br * s.D * 4, cudaMemcpyDeviceToHost);
    if (Vr && d.Br > 0 && e == cudaSuccess)
        e = cudaMemcpy(Vr, c->base + d.vr_off, (size_t)d.Br * s.D * 4, cudaMemcpyDeviceToHost);
    if (w && d.Br > 0 && e == cudaSuccess)
        e = cudaMemcpy(w, c->base + d.w_off, (size_t)d.Br * 4, cudaMemcpyDeviceToHost);
    if (counters && e == cudaSuccess) {
        UnitCounters uc;
        e = cudaMemcpy(&uc, c->base + c->lay.counters + (size_t)d.unit * sizeof(UnitCounters),
                       sizeof(uc), cudaMemcpyDeviceToHost);
        counters[0] = uc.n_live;
        counters[1] = uc.n_res;
        counters[2] = uc.T;
    }
    return cuda_status(e);
}

zsm_status_t zsm_cache_import_unit(zsm_cache_t *c, int32_t layer, int32_t b, int32_t h,
                                   const float *K, const float *V, const float *score,
                                   const int32_t *pos, const float *Kr, const float *Vr,
                                   const uint32_t *w, const int32_t *counters,
                                   zsm_stream_t stream) {
    if (!c || layer < 0 || layer >= c->s.L || b < 0 || b >= c->s.B || h < 0 || h >= c->s.Hkv)
        return ZSM_ERR_INVALID_ARG;
    if (!K || !V || !score || !pos || !counters) return ZSM_ERR_INVALID_ARG;
    const Shape &s = c->s;
    const UnitDesc &d = c->lay.desc[(layer * s.B + b) * s.Hkv + h];
    const size_t cap = (size_t)d.Bp + d.Bc;
    if (d.Br > 0 && (!Kr || !Vr || !w)) return ZSM_ERR_INVALID_ARG;
    if (counters[0] < 0 || (size_t)counters[0] > cap || counters[1] < 0 || counters[1] > d.Br ||
        counters[2] < counters[0])
        return ZSM_ERR_INVALID_ARG;
    for (int32_t i = 0; i < counters[0]; ++i)
        if (std::isnan(score[i])) return ZSM_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(cs) != cudaSuccess) return ZSM_ERR_CUDA;
    c->wrote_everywhere();
    std::vector<uint8_t> raw(cap * s.row_bytes);
    cudaError_t e = cudaSuccess;
    for (int which = 0; which < 2 && e == cudaSuccess; ++which) {
        const float *src = which ? V : K;
        if (s.dtype == ZSM_F32) {
            std::memcpy(raw.data(), src, raw.size());
        } else {
            uint16_t *hd = reinterpret_cast<uint16_t *>(raw.data());
            for (size_t i = 0; i < cap * s.D; ++i) hd[i] = float_to_half_bits(src[i], s.dtype);
        }
        e = cudaMemcpy(c->base + (which ? d.v_off : d.k_off), raw.data(), raw.size(),
                       cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess) e = cudaMemcpy(c->base + d.score_off, score, cap * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(c->base + d.pos_off, pos, cap * 4, cudaMemcpyHostToDevice);
    if (d.Br > 0) {
        if (e == cudaSuccess)
            e = cudaMemcpy(c->base + d.kr_off, Kr, (size_t)d.Br * s.D * 4, cudaMemcpyHostToDevice);
        if (e == cudaSuccess)
            e = cudaMemcpy(c->base + d.vr_off, Vr, (size_t)d.Br * s.D * 4, cudaMemcpyHostToDevice);
        if (e == cudaSuccess)
            e = cudaMemcpy(c->base + d.w_off, w, (size_t)d.Br * 4, cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess) {
        UnitCounters uc;
        uc.n_live = counters[0];
        uc.n_res = counters[1];
        uc.T = counters[2];
        uc.pad = 0;
        e = cudaMemcpy(c->base + c->lay.counters + (size_t)d.unit * sizeof(UnitCounters), &uc,
                       sizeof(uc), cudaMemcpyHostToDevice);
    }
    return cuda_status(e);
}

zsm_status_t zsm_selftest_wait_timeout(zsm_cache_t *c, uint32_t limit_us, zsm_stream_t stream) {
    if (!c || limit_us < 1u || limit_us > 1000000u) return ZSM_ERR_INVALID_ARG;
    const int rc = launch_wait_selftest(reinterpret_cast<int32_t *>(c->base + c->lay.status),
                                        limit_us, static_cast<cudaStream_t>(stream));
    return rc == 0 ? ZSM_OK : ZSM_ERR_CUDA;
}

zsm_status_t zsm_last_device_status(zsm_cache_t *c, zsm_stream_t stream) {
    if (!c) return ZSM_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(cs) != cudaSuccess) return ZSM_ERR_CUDA;
    int32_t st[4] = {0, 0, 0, 0};
    if (cudaMemcpy(st, c->base + c->lay.status, sizeof(st), cudaMemcpyDeviceToHost) != cudaSuccess)
        return ZSM_ERR_CUDA;
    if (st[0] != 0) {
        int32_t zero[4] = {0, 0, 0, 0};
        if (cudaMemcpy(c->base + c->lay.status, zero, sizeof(zero), cudaMemcpyHostToDevice) !=
            cudaSuccess)
            return ZSM_ERR_CUDA;
    }
    if (st[0] == DEV_ERR_CHECK) return ZSM_ERR_DEVICE_CHECK;
    if (st[0] == DEV_ERR_TIMEOUT) return ZSM_ERR_TIMEOUT;
    return st[0] == 0 ? ZSM_OK : ZSM_ERR_DEVICE_CHECK;
}

}  // extern "C"
