// Fused decode step of the budgeted KV cache (Algorithm 1 + Eq. (att_score2)).
//
// Persistent CTAs (two per SM by default) each walk a static list of units.  A producer warp
// streams each unit's arrays through a ring of 16 KiB shared-memory stages with
// 1-D bulk copies (cp.async.bulk + mbarrier); it runs ahead across units, so the
// tail of one unit (softmax, victim search, merge) overlaps the next unit's loads.
// Consumer warps take the tiles in order:
//
//   header   counters, q (G heads), k_new, v_new, fusion counts w
//   K tiles  logits q.k/sqrt(d) of every live token slot          (D1)
//   Kr tiles logits of the merged slots, + alpha*ln w             (D1, Eq. (att_score2))
//   -- softmax over slots + new token                             (D2)
//   meta     score, pos: s <- lambda*s + mean_g a_hat; running argmin of
//            (s, pos) over slots that left the proximity window   (D4, D5)
//   -- residual target: fill, or argmax_r k_r.k_victim and the incremental mean (D6)
//   V tiles, Vr tiles   o = sum a_hat v                            (D3)
//   -- write o; new token into the victim's slot; merged rows; counters (D6, D7)
//
// K and V rows cross HBM exactly once per step; grouped query heads share them.
#include "zsm_decode.cuh"

namespace zsm {

namespace {

constexpr int kMaxThreads = (kMaxConsumerWarps + 1) * 32;

// "where" codes recorded with a timeout
enum : int32_t { W_PRODUCER = 1, W_HEADER = 2, W_K = 3, W_KR = 4, W_META = 5, W_V = 6, W_VR = 7 };

template <int LANES>
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
    for (int off = LANES / 2; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(kMaxThreads, 1) decode_fused_kernel(const DecodeParams p) {
    using E = Elem<T>;
    constexpr int EPL = E::EPL;               // elements per 16-byte lane load
    constexpr int ROWB = D * (int)sizeof(T);  // bytes per token row
    constexpr int LPR = D / EPL;              // lanes per token row
    constexpr int RPW = 32 / LPR;             // token rows per warp-wide load
    constexpr int R = kTileBytes / ROWB;      // token rows per tile
    constexpr int ROWB32 = D * 4;             // residual rows are fp32
    constexpr int LPR32 = D / 4;
    constexpr int RPW32 = 32 / LPR32;
    constexpr int R32 = kTileBytes / ROWB32;
    constexpr int RM = kTileBytes / 8;        // (score, pos) entries per meta tile
    constexpr int HDR_D = 16;                 // unit descriptor
    constexpr int HDR_Q = HDR_D + (int)sizeof(UnitDesc);
    constexpr int HDR_K = HDR_Q + G * ROWB;
    constexpr int HDR_V = HDR_K + ROWB;
    constexpr int HDR_W = HDR_V + ROWB;
    constexpr int UB = 4;                     // row groups in flight per warp

    extern __shared__ __align__(128) uint8_t smem[];
    const int NW = (blockDim.x >> 5) - 1;  // consumer warps
    const int NT = NW * 32;
    const int S = p.stages;
    const int LS = p.l_stride;
    const DecodeSmem L = decode_smem_layout(S, G, D, ROWB, LS, p.br_max_pad, NW);

    uint8_t *ring = smem + L.ring;
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + L.bars);
    uint64_t *empty_bar = full_bar + S;
    volatile int32_t *flags = reinterpret_cast<volatile int32_t *>(smem + L.flags);
    volatile int32_t *abort_flag = flags;  // flags[0]
    float *probs = reinterpret_cast<float *>(smem + L.probs);
    float *qf = reinterpret_cast<float *>(smem + L.qf);
    uint4 *kn_raw = reinterpret_cast<uint4 *>(smem + L.kn);
    uint4 *vn_raw = reinterpret_cast<uint4 *>(smem + L.vn);
    uint32_t *w_s = reinterpret_cast<uint32_t *>(smem + L.w);
    float *opart = reinterpret_cast<float *>(smem + L.opart);
    float *redf = reinterpret_cast<float *>(smem + L.redf);
    float *redf2 = redf + kMaxConsumerWarps * 8;
    uint64_t *red64 = reinterpret_cast<uint64_t *>(smem + L.red64);
    float *dots = reinterpret_cast<float *>(smem + L.dots);
    float *kc = reinterpret_cast<float *>(smem + L.rows);
    float *vc = kc + D;
    float *mk = vc + D;
    float *mv = mk + D;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], NW);
        }
        flags[0] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const int first = p.sched_off[blockIdx.x];
    const int last = p.sched_off[blockIdx.x + 1];

    // =====================================================================
    // Producer: one thread issues every bulk copy of this CTA.
    // =====================================================================
    if (warp == NW) {
        if (lane != 0 || first >= last) return;
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        auto acquire = [&](uint32_t bytes, uint64_t *&bar) -> uint8_t * {
            if (!mbar_wait_bounded(&empty_bar[s], ph ^ 1u, abort_flag, p.status, W_PRODUCER)) {
                ok = false;
                return nullptr;
            }
            bar = &full_bar[s];
            mbar_arrive_expect_tx(bar, bytes);
            uint8_t *dst = ring + static_cast<size_t>(s) * kTileBytes;
            if (++s == S) {
                s = 0;
                ph ^= 1u;
            }
            return dst;
        };
        auto load_desc = [&](int i) -> UnitDesc {
            UnitDesc d;
            const uint4 *src = reinterpret_cast<const uint4 *>(p.sched_desc + i);
            uint4 *dst = reinterpret_cast<uint4 *>(&d);
#pragma unroll
            for (int k = 0; k < 5; ++k) dst[k] = __ldg(src + k);
            return d;
        };
        auto load_cnt = [&](int unit) -> int4 {
            return *reinterpret_cast<const int4 *>(p.counters + unit);
        };

        // descriptors are fetched two units ahead, counters one unit ahead
        UnitDesc d_cur = load_desc(first);
        int4 c_cur = load_cnt(d_cur.unit);
        UnitDesc d_nxt = d_cur;
        if (first + 1 < last) d_nxt = load_desc(first + 1);

        for (int i = first; i < last && ok; ++i) {
            int4 c_nxt = c_cur;
            UnitDesc d_nx2 = d_nxt;
            if (i + 1 < last) c_nxt = load_cnt(d_nxt.unit);
            if (i + 2 < last) d_nx2 = load_desc(i + 2);

            const UnitDesc &d = d_cur;
            const int cap = d.Bp + d.Bc;
            const int n_live = min(max(c_cur.x, 0), cap);
            const int n_res = min(max(c_cur.y, 0), d.Br);
            const int ul = d.unit - p.unit_base;
            const int br_pad = (d.Br + 3) & ~3;
            uint64_t *bar = nullptr;
            uint8_t *dst;

            // header
            dst = acquire(HDR_W + br_pad * 4u, bar);
            if (!ok) break;
            bulk_g2s(dst, p.counters + d.unit, 16u, bar);
            bulk_g2s(dst + HDR_D, p.sched_desc + i, (uint32_t)sizeof(UnitDesc), bar);
            bulk_g2s(dst + HDR_Q, static_cast<const uint8_t *>(p.q) + (size_t)ul * G * ROWB,
                     G * ROWB, bar);
            bulk_g2s(dst + HDR_K, static_cast<const uint8_t *>(p.k_new) + (size_t)ul * ROWB, ROWB,
                     bar);
            bulk_g2s(dst + HDR_V, static_cast<const uint8_t *>(p.v_new) + (size_t)ul * ROWB, ROWB,
                     bar);
            if (br_pad > 0) bulk_g2s(dst + HDR_W, p.base + d.w_off, br_pad * 4u, bar);

            // K token rows, then residual K rows
            for (int r0 = 0; r0 < n_live && ok; r0 += R) {
                const uint32_t bytes = static_cast<uint32_t>(min(R, n_live - r0)) * ROWB;
                dst = acquire(bytes, bar);
                if (ok) bulk_g2s(dst, p.base + d.k_off + (size_t)r0 * ROWB, bytes, bar);
            }
            for (int r0 = 0; r0 < n_res && ok; r0 += R32) {
                const uint32_t bytes = static_cast<uint32_t>(min(R32, n_res - r0)) * ROWB32;
                dst = acquire(bytes, bar);
                if (ok) bulk_g2s(dst, p.base + d.kr_off + (size_t)r0 * ROWB32, bytes, bar);
            }
            // scores and positions
            for (int j0 = 0; j0 < n_live && ok; j0 += RM) {
                const uint32_t n4 = static_cast<uint32_t>((min(RM, n_live - j0) + 3) & ~3);
                dst = acquire(n4 * 8u, bar);
                if (ok) {
                    bulk_g2s(dst, p.base + d.score_off + (size_t)j0 * 4, n4 * 4u, bar);
                    bulk_g2s(dst + RM * 4, p.base + d.pos_off + (size_t)j0 * 4, n4 * 4u, bar);
                }
            }
            // V token rows, then residual V rows
            for (int r0 = 0; r0 < n_live && ok; r0 += R) {
                const uint32_t bytes = static_cast<uint32_t>(min(R, n_live - r0)) * ROWB;
                dst = acquire(bytes, bar);
                if (ok) bulk_g2s(dst, p.base + d.v_off + (size_t)r0 * ROWB, bytes, bar);
            }
            for (int r0 = 0; r0 < n_res && ok; r0 += R32) {
                const uint32_t bytes = static_cast<uint32_t>(min(R32, n_res - r0)) * ROWB32;
                dst = acquire(bytes, bar);
                if (ok) bulk_g2s(dst, p.base + d.vr_off + (size_t)r0 * ROWB32, bytes, bar);
            }
            d_cur = d_nxt;
            d_nxt = d_nx2;
            c_cur = c_nxt;
        }
        if (!ok) {
            // give copies already in flight time to land before the CTA's memory goes away
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
        return;
    }

    // =====================================================================
    // Consumers
    // =====================================================================
    const int l = lane % LPR;      // 16-byte column of a token row
    const int sub = lane / LPR;    // which of the RPW rows of a warp-wide load
    const int l32 = lane % LPR32;  // same for fp32 residual rows
    const int sub32 = lane / LPR32;

    int cs = 0;
    uint32_t cph = 0;
    auto wait_full = [&](int where) -> const uint8_t * {
        if (!mbar_wait_bounded(&full_bar[cs], cph, abort_flag, p.status, where)) return nullptr;
        return ring + static_cast<size_t>(cs) * kTileBytes;
    };
    auto release = [&]() {
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[cs]);
        if (++cs == S) {
            cs = 0;
            cph ^= 1u;
        }
    };
    auto csync = [&]() { named_bar_sync(1, NT); };

    for (int i = first; i < last; ++i) {
        // ---------------- header ----------------
        const uint8_t *h = wait_full(W_HEADER);
        if (!h) return;
        const int4 cnt = *reinterpret_cast<const int4 *>(h);
        const UnitDesc d = *reinterpret_cast<const UnitDesc *>(h + HDR_D);
        const int cap = d.Bp + d.Bc;
        const int ul = d.unit - p.unit_base;
        const int br_pad = (d.Br + 3) & ~3;
        if (tid == 0 && (cnt.x < 0 || cnt.x > cap || cnt.y < 0 || cnt.y > d.Br))
            dev_set_status(p.status, DEV_ERR_CHECK, d.unit, 1);
        const int n_live = min(max(cnt.x, 0), cap);
        const int n_res = min(max(cnt.y, 0), d.Br);
        const int Tpos = cnt.z;
        const int n_ent = n_live + n_res + 1;

        float qreg[G][EPL];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const uint4 raw = *reinterpret_cast<const uint4 *>(h + HDR_Q + g * ROWB + l * 16);
            E::widen(raw, qreg[g]);
        }
        {
            const T *qs = reinterpret_cast<const T *>(h + HDR_Q);
            for (int k = tid; k < G * D; k += NT) qf[k] = E::to_float(qs[k]);
            const uint4 *ks = reinterpret_cast<const uint4 *>(h + HDR_K);
            const uint4 *vs = reinterpret_cast<const uint4 *>(h + HDR_V);
            for (int k = tid; k < ROWB / 16; k += NT) {
                kn_raw[k] = ks[k];
                vn_raw[k] = vs[k];
            }
            const uint32_t *ws = reinterpret_cast<const uint32_t *>(h + HDR_W);
            for (int k = tid; k < br_pad; k += NT) w_s[k] = ws[k];
        }
        release();

        // ---------------- D1: logits of the token slots ----------------
        for (int r0 = 0; r0 < n_live; r0 += R) {
            const uint8_t *tile = wait_full(W_K);
            if (!tile) return;
            const int rows = min(R, n_live - r0);
            for (int base = warp * RPW; base < rows; base += NW * RPW * UB) {
                uint4 raw[UB];
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    const int row = base + u * NW * RPW + sub;
                    raw[u] = row < rows
                                 ? *reinterpret_cast<const uint4 *>(tile + row * ROWB + l * 16)
                                 : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    const int row = base + u * NW * RPW + sub;
                    float f[EPL];
                    E::widen(raw[u], f);
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        float acc = 0.f;
#pragma unroll
                        for (int e = 0; e < EPL; ++e) acc = fmaf(qreg[g][e], f[e], acc);
                        acc = group_sum<LPR>(acc);
                        if (l == 0 && row < rows) probs[g * LS + r0 + row] = acc * p.scale;
                    }
                }
            }
            release();
        }
        csync();  // qf, kn_raw, w_s of this unit are in place

        // ---------------- D1: logits of the merged slots, + alpha ln w ----------------
        for (int r0 = 0; r0 < n_res; r0 += R32) {
            const uint8_t *tile = wait_full(W_KR);
            if (!tile) return;
            const int rows = min(R32, n_res - r0);
            for (int base = warp * RPW32; base < rows; base += NW * RPW32) {
                const int row = base + sub32;
                float4 kr = make_float4(0.f, 0.f, 0.f, 0.f);
                if (row < rows)
                    kr = *reinterpret_cast<const float4 *>(tile + row * ROWB32 + l32 * 16);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float4 qv = *reinterpret_cast<const float4 *>(qf + g * D + l32 * 4);
                    float acc = qv.x * kr.x;
                    acc = fmaf(qv.y, kr.y, acc);
                    acc = fmaf(qv.z, kr.z, acc);
                    acc = fmaf(qv.w, kr.w, acc);
                    acc = group_sum<LPR32>(acc);
                    if (l32 == 0 && row < rows)
                        probs[g * LS + n_live + r0 + row] =
                            fmaf(p.alpha, logf(static_cast<float>(w_s[r0 + row])), acc * p.scale);
                }
            }
            release();
        }
        // logit of the new token itself
        if (warp == NW - 1) {
            float f[EPL];
            E::widen(sub == 0 ? kn_raw[l] : make_uint4(0, 0, 0, 0), f);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float *qg = qf + g * D + l * EPL;
                float acc = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) acc = fmaf(qg[e], f[e], acc);
                acc = group_sum<32>(acc);
                if (lane == 0) probs[g * LS + n_ent - 1] = acc * p.scale;
            }
        }
        csync();

        // ---------------- D2: softmax over slots + new token ----------------
        float mx[G], inv[G];
#pragma unroll
        for (int g = 0; g < G; ++g) mx[g] = -INFINITY;
        for (int j = tid; j < n_ent; j += NT) {
#pragma unroll
            for (int g = 0; g < G; ++g) mx[g] = fmaxf(mx[g], probs[g * LS + j]);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1)
                mx[g] = fmaxf(mx[g], __shfl_xor_sync(0xffffffffu, mx[g], off));
            if (lane == 0) redf[warp * G + g] = mx[g];
        }
        csync();
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float m = redf[g];
            for (int wv = 1; wv < NW; ++wv) m = fmaxf(m, redf[wv * G + g]);
            mx[g] = m;
        }
        {
            float sm[G];
#pragma unroll
            for (int g = 0; g < G; ++g) sm[g] = 0.f;
            for (int j = tid; j < n_ent; j += NT) {
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float e = expf(probs[g * LS + j] - mx[g]);
                    probs[g * LS + j] = e;
                    sm[g] += e;
                }
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                sm[g] = group_sum<32>(sm[g]);
                if (lane == 0) redf2[warp * G + g] = sm[g];
            }
        }
        csync();
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float z = redf2[g];
            for (int wv = 1; wv < NW; ++wv) z += redf2[wv * G + g];
            inv[g] = 1.0f / z;
        }

        // ---------------- D4 + D5: score update and victim search ----------------
        const bool evict = (n_live == cap);  // the new token does not fit: Alg. 1 l.7-11
        const int cut = Tpos - d.Bp;         // positions <= cut have left the proximity window
        float *score_g = reinterpret_cast<float *>(p.base + d.score_off);
        int32_t *pos_g = reinterpret_cast<int32_t *>(p.base + d.pos_off);
        uint64_t best = ~0ull;
        int best_slot = -1;
        for (int j0 = 0; j0 < n_live; j0 += RM) {
            const uint8_t *tile = wait_full(W_META);
            if (!tile) return;
            const int n = min(RM, n_live - j0);
            const float *ts = reinterpret_cast<const float *>(tile);
            const int32_t *tp = reinterpret_cast<const int32_t *>(tile + RM * 4);
            for (int k = tid; k < n; k += NT) {
                float a = 0.f;
#pragma unroll
                for (int g = 0; g < G; ++g) a += probs[g * LS + j0 + k] * inv[g];
                a *= (1.0f / G);
                const float s_new = fmaf(p.lambda, ts[k], a);  // Eq. (score)
                score_g[j0 + k] = s_new;
                const int32_t pj = tp[k];
                if (evict && pj <= cut) {
                    const uint64_t key =
                        (static_cast<uint64_t>(__float_as_uint(s_new)) << 32) | (uint32_t)pj;
                    if (key < best) {
                        best = key;
                        best_slot = j0 + k;
                    }
                }
            }
            release();
        }
        float s_tok = 0.f;  // first score of the new token: its own attention weight
#pragma unroll
        for (int g = 0; g < G; ++g) s_tok += probs[g * LS + n_ent - 1] * inv[g];
        s_tok *= (1.0f / G);

        int victim_slot = -1;  // >= 0: token slot; -2: the new token itself (B_p = 0)
        int victim_pos = -1;
        if (evict) {
            if (tid == 0 && d.Bp == 0) {
                const uint64_t key =
                    (static_cast<uint64_t>(__float_as_uint(s_tok)) << 32) | (uint32_t)Tpos;
                if (key < best) {
                    best = key;
                    best_slot = -2;
                }
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
                const uint64_t ob = __shfl_xor_sync(0xffffffffu, best, off);
                const int os = __shfl_xor_sync(0xffffffffu, best_slot, off);
                if (ob < best) {
                    best = ob;
                    best_slot = os;
                }
            }
            if (lane == 0) {
                red64[warp * 2] = best;
                red64[warp * 2 + 1] = static_cast<uint64_t>(static_cast<uint32_t>(best_slot));
            }
            csync();
            best = red64[0];
            best_slot = static_cast<int>(static_cast<uint32_t>(red64[1]));
            for (int wv = 1; wv < NW; ++wv) {
                const uint64_t ob = red64[wv * 2];
                if (ob < best) {
                    best = ob;
                    best_slot = static_cast<int>(static_cast<uint32_t>(red64[wv * 2 + 1]));
                }
            }
            if (best == ~0ull) {
                if (tid == 0) dev_set_status(p.status, DEV_ERR_CHECK, d.unit, 2);
            } else {
                victim_slot = best_slot;
                victim_pos = static_cast<int>(static_cast<uint32_t>(best & 0xffffffffull));
            }
        }
        const bool have_victim = evict && victim_slot != -1;

        // ---------------- D6: where the victim goes ----------------
        int merge_slot = -1;  // report: slot merged into, -2 fill, -1 none
        int res_target = -1;  // residual row to write after the V pass
        uint32_t res_w = 0;
        if (have_victim && d.Br > 0) {
            if (warp == 0) {
                for (int k = lane; k < LPR; k += 32) {
                    float f[EPL];
                    const uint4 raw = victim_slot >= 0
                                          ? *reinterpret_cast<const uint4 *>(
                                                p.base + d.k_off + (size_t)victim_slot * ROWB + k * 16)
                                          : kn_raw[k];
                    E::widen(raw, f);
#pragma unroll
                    for (int e = 0; e < EPL; ++e) kc[k * EPL + e] = f[e];
                }
            }
            if (warp == (NW > 1 ? 1 : 0)) {
                for (int k = lane; k < LPR; k += 32) {
                    float f[EPL];
                    const uint4 raw = victim_slot >= 0
                                          ? *reinterpret_cast<const uint4 *>(
                                                p.base + d.v_off + (size_t)victim_slot * ROWB + k * 16)
                                          : vn_raw[k];
                    E::widen(raw, f);
#pragma unroll
                    for (int e = 0; e < EPL; ++e) vc[k * EPL + e] = f[e];
                }
            }
            csync();
            const float *Kr_g = reinterpret_cast<const float *>(p.base + d.kr_off);
            const float *Vr_g = reinterpret_cast<const float *>(p.base + d.vr_off);
            if (n_res < d.Br) {
                // Alg. 1 l.12-13: a free residual slot takes the token as it is
                res_target = n_res;
                res_w = 1;
                merge_slot = -2;
                for (int k = tid; k < D; k += NT) {
                    mk[k] = kc[k];
                    mv[k] = vc[k];
                }
            } else {
                // Eq. (hatr): raw dot product with every merged key
                for (int r = warp; r < n_res; r += NW) {
                    float acc = 0.f;
                    for (int k = lane; k < LPR32; k += 32) {
                        const float4 kr = *reinterpret_cast<const float4 *>(Kr_g + (size_t)r * D + k * 4);
                        acc = fmaf(kr.x, kc[k * 4 + 0], acc);
                        acc = fmaf(kr.y, kc[k * 4 + 1], acc);
                        acc = fmaf(kr.z, kc[k * 4 + 2], acc);
                        acc = fmaf(kr.w, kc[k * 4 + 3], acc);
                    }
                    acc = group_sum<32>(acc);
                    if (lane == 0) dots[r] = acc;
                }
                csync();
                if (warp == 0) {
                    float bd = -INFINITY;
                    int br = 0x7fffffff;
                    for (int r = lane; r < n_res; r += 32) {
                        const float dv = dots[r];
                        if (br == 0x7fffffff || dv > bd) {
                            bd = dv;
                            br = r;
                        }
                    }
#pragma unroll
                    for (int off = 16; off >= 1; off >>= 1) {
                        const float od = __shfl_xor_sync(0xffffffffu, bd, off);
                        const int orr = __shfl_xor_sync(0xffffffffu, br, off);
                        if (orr != 0x7fffffff && (br == 0x7fffffff || od > bd || (od == bd && orr < br))) {
                            bd = od;
                            br = orr;
                        }
                    }
                    if (lane == 0) flags[2] = br;
                }
                csync();
                res_target = flags[2];
                merge_slot = res_target;
                const uint32_t wr_u = w_s[res_target];
                res_w = wr_u + 1u;
                const float wr = static_cast<float>(wr_u);
                // Eq. (kvr): incremental mean of key and value
                for (int k = tid; k < D; k += NT) {
                    mk[k] = fmaf(wr, Kr_g[(size_t)res_target * D + k], kc[k]) / (wr + 1.0f);
                    mv[k] = fmaf(wr, Vr_g[(size_t)res_target * D + k], vc[k]) / (wr + 1.0f);
                }
            }
        }

        // ---------------- D3: output ----------------
        float acc[G][EPL];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[g][e] = 0.f;
        for (int r0 = 0; r0 < n_live; r0 += R) {
            const uint8_t *tile = wait_full(W_V);
            if (!tile) return;
            const int rows = min(R, n_live - r0);
            for (int base = warp * RPW; base < rows; base += NW * RPW * UB) {
                uint4 raw[UB];
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    const int row = base + u * NW * RPW + sub;
                    raw[u] = row < rows
                                 ? *reinterpret_cast<const uint4 *>(tile + row * ROWB + l * 16)
                                 : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    const int row = base + u * NW * RPW + sub;
                    float f[EPL];
                    E::widen(raw[u], f);
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const float pj = row < rows ? probs[g * LS + r0 + row] : 0.f;
#pragma unroll
                        for (int e = 0; e < EPL; ++e) acc[g][e] = fmaf(pj, f[e], acc[g][e]);
                    }
                }
            }
            release();
        }
        float acc32[G][4];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc32[g][e] = 0.f;
        for (int r0 = 0; r0 < n_res; r0 += R32) {
            const uint8_t *tile = wait_full(W_VR);
            if (!tile) return;
            const int rows = min(R32, n_res - r0);
            for (int base = warp * RPW32; base < rows; base += NW * RPW32) {
                const int row = base + sub32;
                if (row < rows) {
                    const float4 vr = *reinterpret_cast<const float4 *>(tile + row * ROWB32 + l32 * 16);
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const float pj = probs[g * LS + n_live + r0 + row];
                        acc32[g][0] = fmaf(pj, vr.x, acc32[g][0]);
                        acc32[g][1] = fmaf(pj, vr.y, acc32[g][1]);
                        acc32[g][2] = fmaf(pj, vr.z, acc32[g][2]);
                        acc32[g][3] = fmaf(pj, vr.w, acc32[g][3]);
                    }
                }
            }
            release();
        }
        // fold the RPW row groups of a warp, then the warps
#pragma unroll
        for (int g = 0; g < G; ++g) {
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                float v = acc[g][e];
#pragma unroll
                for (int off = LPR; off < 32; off <<= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
                if (sub == 0) opart[(warp * G + g) * D + l * EPL + e] = v;
            }
        }
        __syncwarp();
        if (n_res > 0) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float v = acc32[g][e];
#pragma unroll
                    for (int off = LPR32; off < 32; off <<= 1)
                        v += __shfl_xor_sync(0xffffffffu, v, off);
                    if (sub32 == 0) opart[(warp * G + g) * D + l32 * 4 + e] += v;
                }
            }
        }
        csync();
        {
            const T *vn = reinterpret_cast<const T *>(vn_raw);
            T *out = static_cast<T *>(p.out) + (size_t)ul * G * D;
            for (int k = tid; k < G * D; k += NT) {
                const int g = k / D, dim = k % D;
                float sum = 0.f;
                for (int wv = 0; wv < NW; ++wv) sum += opart[(wv * G + g) * D + dim];
                sum = fmaf(probs[g * LS + n_ent - 1], E::to_float(vn[dim]), sum);
                out[k] = E::from_float(sum * inv[g]);
            }
        }

        // ---------------- D6 + D7: write-back (every read of this unit is done) ----------------
        const bool insert = evict ? (have_victim && victim_slot >= 0) : true;
        const int ins_slot = evict ? victim_slot : n_live;
        if (insert) {
            if (tid < ROWB / 16) {
                reinterpret_cast<uint4 *>(p.base + d.k_off + (size_t)ins_slot * ROWB)[tid] = kn_raw[tid];
            } else if (tid < 2 * (ROWB / 16)) {
                const int k = tid - ROWB / 16;
                reinterpret_cast<uint4 *>(p.base + d.v_off + (size_t)ins_slot * ROWB)[k] = vn_raw[k];
            }
        }
        if (res_target >= 0) {
            float *Kr_g = reinterpret_cast<float *>(p.base + d.kr_off);
            float *Vr_g = reinterpret_cast<float *>(p.base + d.vr_off);
            for (int k = tid; k < D; k += NT) {
                Kr_g[(size_t)res_target * D + k] = mk[k];
                Vr_g[(size_t)res_target * D + k] = mv[k];
            }
        }
        if (tid == 0) {
            if (insert) {
                score_g[ins_slot] = s_tok;
                pos_g[ins_slot] = Tpos;
            }
            if (res_target >= 0)
                reinterpret_cast<uint32_t *>(p.base + d.w_off)[res_target] = res_w;
            UnitCounters c;
            c.n_live = n_live + ((!evict) ? 1 : 0);
            c.n_res = n_res + ((merge_slot == -2) ? 1 : 0);
            c.T = Tpos + 1;
            c.pad = 0;
            *reinterpret_cast<int4 *>(p.counters + d.unit) = *reinterpret_cast<int4 *>(&c);
            if (p.victim_pos) p.victim_pos[ul] = victim_pos;
            if (p.merge_slot) p.merge_slot[ul] = merge_slot;
        }
        csync();  // shared scratch is free for the next unit
    }
}

template <typename T, int D, int G>
int launch_one(const DecodeParams &p, int grid, int consumer_warps, cudaStream_t stream) {
    const int threads = (consumer_warps + 1) * 32;
    const DecodeSmem L = decode_smem_layout(p.stages, G, D, D * (int)sizeof(T), p.l_stride,
                                            p.br_max_pad, consumer_warps);
    decode_fused_kernel<T, D, G><<<grid, threads, L.total, stream>>>(p);
    return static_cast<int>(cudaGetLastError());
}

template <typename T, int D, int G>
int prepare_one(int smem_bytes, int threads, int *max_ctas) {
    cudaError_t e = cudaFuncSetAttribute(decode_fused_kernel<T, D, G>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return static_cast<int>(e);
    int n = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_fused_kernel<T, D, G>, threads,
                                                      smem_bytes);
    if (max_ctas) *max_ctas = n;
    return static_cast<int>(e);
}

#define ZSM_DISPATCH(FN, ...)                                                         \
    do {                                                                              \
        if (dtype == 0) {                                                             \
            if (D == 64) ZSM_DISPATCH_G(FN, float, 64, __VA_ARGS__);                  \
            if (D == 128) ZSM_DISPATCH_G(FN, float, 128, __VA_ARGS__);                \
        } else if (dtype == 1) {                                                      \
            if (D == 64) ZSM_DISPATCH_G(FN, __half, 64, __VA_ARGS__);                 \
            if (D == 128) ZSM_DISPATCH_G(FN, __half, 128, __VA_ARGS__);               \
        } else if (dtype == 2) {                                                      \
            if (D == 64) ZSM_DISPATCH_G(FN, __nv_bfloat16, 64, __VA_ARGS__);          \
            if (D == 128) ZSM_DISPATCH_G(FN, __nv_bfloat16, 128, __VA_ARGS__);        \
        }                                                                             \
    } while (0)

#define ZSM_DISPATCH_G(FN, TT, DD, ...)                      \
    do {                                                     \
        if (G == 1) return FN<TT, DD, 1>(__VA_ARGS__);       \
        if (G == 2) return FN<TT, DD, 2>(__VA_ARGS__);       \
        if (G == 4) return FN<TT, DD, 4>(__VA_ARGS__);       \
        if (G == 8) return FN<TT, DD, 8>(__VA_ARGS__);       \
    } while (0)

}  // namespace

int launch_decode_fused(int dtype, int D, int G, const DecodeParams &p, int grid,
                        int consumer_warps, cudaStream_t stream) {
    ZSM_DISPATCH(launch_one, p, grid, consumer_warps, stream);
    return -1;
}

int prepare_decode_fused(int dtype, int D, int G, int smem_bytes, int threads,
                         int *max_ctas_per_sm) {
    ZSM_DISPATCH(prepare_one, smem_bytes, threads, max_ctas_per_sm);
    return -1;
}

}  // namespace zsm
