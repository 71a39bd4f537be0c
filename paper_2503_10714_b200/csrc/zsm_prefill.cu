// One-shot compression of a prompt's K/V into the per-head budgets.
//
//   P1  scores from the prompt's last W queries: causal softmax rows combined by
//       Eq. (score) unrolled, s_t = (1/G) sum_g sum_tau lambda^(T-1-tau) a_t^(tau)
//         prefill_logits[_mma]  scaled, masked q.k into scratch + per-chunk (max, sum exp);
//                          16-bit storage: on the tensor cores
//         prefill_rowstat  per query row: max and weight/sum
//         prefill_scores   s_t = sum_rows exp(logit - max) * weight/sum
//   P2  the latest B_p positions are kept as they are (Sec. 3.2)
//   P3  prefill_select     of the rest, the B_c highest (score, position) stay: radix
//                          select of the eviction threshold, then ordered compaction
//   P4  prefill_merge[_rows] evicted tokens, ascending position, fill-or-merge into the
//                          residual slots (Alg. 1 fill/merge branch, Eq. (hatr), (kvr));
//                          the row-per-warp form holds the merged rows in registers (B_r <= 128)
//   P5  prefill_gather     survivors' rows, scores and positions into the unit's slots
#include "zsm_prefill.cuh"
#include "zsm_prefill_full.cuh"

#include <algorithm>

namespace zsm {

namespace {

// ---------------------------------------------------------------------------
// P1a: logits of one chunk of prompt positions against every window query.
// grid (chunks, units), 256 threads: thread (tx, ty) owns positions tx+32i and
// query rows ty*4+j of the current block of 32 query rows.
// ---------------------------------------------------------------------------
constexpr int kQB = 32;  // query rows per pass

template <typename T, int D>
__global__ void __launch_bounds__(256) prefill_logits_kernel(const PrefillParams p) {
    using E = Elem<T>;
    constexpr int CH = kPrefillChunk;
    constexpr int LD = D + 4;  // padded row, keeps 128-bit shared loads conflict-free
    extern __shared__ __align__(16) float sm[];
    float *Ks = sm;            // [CH][LD]
    float *Qs = sm + CH * LD;  // [kQB][LD]

    const int ul = blockIdx.y;
    const int b = ul / p.n_kv_heads, h = ul % p.n_kv_heads;
    const int t0 = blockIdx.x * CH;
    const int T_len = p.T, W = p.W, G = p.G, GW = p.G * p.W;
    const int n_chunks = gridDim.x;
    const int tid = threadIdx.x, tx = tid & 31, ty = tid >> 5;
    const T *Kg = static_cast<const T *>(p.K) + ((size_t)ul * T_len) * D;
    const int n_q_heads = p.n_kv_heads * G;

    for (int k = tid; k < CH * (D / 4); k += 256) {
        const int r = k / (D / 4), c = (k % (D / 4)) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (t0 + r < T_len) {
            const T *src = Kg + (size_t)(t0 + r) * D + c;
            v = make_float4(E::to_float(src[0]), E::to_float(src[1]), E::to_float(src[2]),
                            E::to_float(src[3]));
        }
        *reinterpret_cast<float4 *>(Ks + r * LD + c) = v;
    }
    float *logits = reinterpret_cast<float *>(p.ws + p.wl.logits) + (size_t)ul * GW * T_len;
    float2 *partial = reinterpret_cast<float2 *>(p.ws + p.wl.partial) + (size_t)ul * GW * n_chunks;

    for (int qb = 0; qb < GW; qb += kQB) {
        __syncthreads();
        for (int k = tid; k < kQB * (D / 4); k += 256) {
            const int r = k / (D / 4), c = (k % (D / 4)) * 4;
            const int gw = qb + r;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (gw < GW) {
                const int g = gw / W, wq = gw % W;
                const T *src = static_cast<const T *>(p.Qw) +
                               (((size_t)b * n_q_heads + h * G + g) * W + wq) * D + c;
                v = make_float4(E::to_float(src[0]), E::to_float(src[1]), E::to_float(src[2]),
                                E::to_float(src[3]));
            }
            *reinterpret_cast<float4 *>(Qs + r * LD + c) = v;
        }
        __syncthreads();
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 4
        for (int dd = 0; dd < D; dd += 4) {
            float4 a[4], q4[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                a[i] = *reinterpret_cast<const float4 *>(Ks + (tx + 32 * i) * LD + dd);
#pragma unroll
            for (int j = 0; j < 4; ++j)
                q4[j] = *reinterpret_cast<const float4 *>(Qs + (ty * 4 + j) * LD + dd);
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc[i][j] = fmaf(a[i].x, q4[j].x, acc[i][j]);
                    acc[i][j] = fmaf(a[i].y, q4[j].y, acc[i][j]);
                    acc[i][j] = fmaf(a[i].z, q4[j].z, acc[i][j]);
                    acc[i][j] = fmaf(a[i].w, q4[j].w, acc[i][j]);
                }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gw = qb + ty * 4 + j;
            if (gw >= GW) continue;  // uniform per warp
            const int tau = T_len - W + (gw % W);  // the query's own position: keys 0..tau
            float m = -INFINITY;
            float lg[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int t = t0 + tx + 32 * i;
                lg[i] = (t < T_len && t <= tau) ? acc[i][j] * p.scale : -INFINITY;
                if (t < T_len) logits[(size_t)gw * T_len + t] = lg[i];
                m = fmaxf(m, lg[i]);
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
            float sum = 0.f;
            if (m > -INFINITY) {
#pragma unroll
                for (int i = 0; i < 4; ++i) sum += expf(lg[i] - m);
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
            if (tx == 0) partial[(size_t)gw * n_chunks + blockIdx.x] = make_float2(m, sum);
        }
    }
}

// ---------------------------------------------------------------------------
// P1a on the tensor cores (16-bit storage): the window scoring is a dense
// (G*W) x d x T contraction, 32 flop per K byte at G*W = 32 -- above what plain
// FMAs can do at HBM speed.  Same outputs as prefill_logits_kernel.
// Persistent CTAs, grid (CTAs per unit, units): CTA x of a unit takes the unit's chunks
// x, x + gridDim.x, ...  A producer warp streams the chunks' keys (contiguous in memory:
// one bulk copy per chunk) through a ring of shared-memory stages, so a chunk's load runs
// under the chunks before it; eight consumer warps take a chunk each time: warp w owns its
// positions 16w .. 16w+15, whose A fragments are read once (mma.sync m16n8k16, contraction
// index permuted as in the decode kernel) -- the stage is handed back at once -- and reused
// for every block of eight query rows.  Scaled, masked logits go through a shared tile,
// which gives coalesced row writes and the per-row (max, sum exp) of the chunk.  A window of
// at most 32 query rows (the usual case) is loaded once per CTA, not once per chunk.
// ---------------------------------------------------------------------------
constexpr int kP1Stages = 2;  // two CTAs of two stages per SM: four chunks in flight
constexpr int kP1Threads = 288;  // 8 consumer warps + the producer warp
enum : int32_t { WP1_PRODUCER = 41, WP1_CHUNK = 42 };

template <typename T, int D>
__global__ void __launch_bounds__(kP1Threads) prefill_logits_mma_kernel(const PrefillParams p) {
    static_assert(sizeof(T) == 2, "16-bit storage");
    constexpr int CH = kPrefillChunk;  // 128 positions = 8 warps x 16 rows
    constexpr int ROWB = D * 2;
    constexpr int SEG = ROWB / 64;
    constexpr int LT = CH + 4;         // padded tile row (floats)
    constexpr int STAGE = CH * ROWB;
    extern __shared__ __align__(128) uint8_t smb[];
    uint8_t *Kring = smb;                                        // [stages][CH][ROWB]
    uint8_t *Qs = Kring + kP1Stages * STAGE;                     // [kQB][ROWB] block of queries
    float *lt = reinterpret_cast<float *>(Qs + kQB * ROWB);      // [kQB][LT] logits of the block
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(lt + kQB * LT);
    uint64_t *empty_bar = full_bar + kP1Stages;
    volatile int32_t *abort_flag = reinterpret_cast<volatile int32_t *>(empty_bar + kP1Stages);

    const int ul = blockIdx.y;
    const int b = ul / p.n_kv_heads, h = ul % p.n_kv_heads;
    const int T_len = p.T, W = p.W, G = p.G, GW = p.G * p.W;
    const int n_chunks = (T_len + CH - 1) / CH;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gq = lane >> 2, tig = lane & 3;
    const uint8_t *Kg = static_cast<const uint8_t *>(p.K) + ((size_t)ul * T_len) * ROWB;
    const int n_q_heads = p.n_kv_heads * G;

    if (tid == 0) {
        for (int s = 0; s < kP1Stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 8);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    if (warp == 8) {  // producer
        if (lane != 0) return;
        int s = 0;
        uint32_t ph = 0;
        for (int c = blockIdx.x; c < n_chunks; c += gridDim.x) {
            if (!mbar_wait_bounded(&empty_bar[s], ph ^ 1u, abort_flag, p.status, WP1_PRODUCER)) {
                // copies in flight land in this CTA's memory: wait for them before leaving
                const uint64_t t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
                return;
            }
            const uint32_t bytes = static_cast<uint32_t>(min(CH, T_len - c * CH)) * ROWB;
            mbar_arrive_expect_tx(&full_bar[s], bytes);
            bulk_g2s(Kring + (size_t)s * STAGE, Kg + (size_t)c * CH * ROWB, bytes, &full_bar[s]);
            if (++s == kP1Stages) {
                s = 0;
                ph ^= 1u;
            }
        }
        return;
    }

    auto csync = [&]() { named_bar_sync(1, 256); };
    auto load_queries = [&](int qb) {
        for (int k = tid; k < kQB * (ROWB / 16); k += 256) {
            const int r = k / (ROWB / 16), c = k % (ROWB / 16);
            const int gw = qb + r;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (gw < GW) {
                const int g = gw / W, wq = gw % W;
                v = *reinterpret_cast<const uint4 *>(static_cast<const uint8_t *>(p.Qw) +
                        (((size_t)b * n_q_heads + h * G + g) * W + wq) * ROWB + c * 16);
            }
            *reinterpret_cast<uint4 *>(Qs + r * ROWB + c * 16) = v;
        }
    };
    const bool one_block = GW <= kQB;  // the whole window fits the query block: load it once
    if (one_block) {
        load_queries(0);
        csync();
    }
    float *logits = reinterpret_cast<float *>(p.ws + p.wl.logits) + (size_t)ul * GW * T_len;
    float2 *partial = reinterpret_cast<float2 *>(p.ws + p.wl.partial) + (size_t)ul * GW * n_chunks;

    int cs = 0;
    uint32_t cph = 0;
    for (int chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
        const int t0 = chunk * CH;
        if (!mbar_wait_bounded(&full_bar[cs], cph, abort_flag, p.status, WP1_CHUNK)) return;
        // this warp's 16 positions as A fragments, all segments (kept for every block of query
        // rows); rows past the prompt's end hold leftovers of an earlier chunk: their logits are
        // masked below, never summed
        uint4 fa[SEG], fc[SEG];
        {
            const uint8_t *pa = Kring + (size_t)cs * STAGE + (warp * 16 + gq) * ROWB + tig * 16;
#pragma unroll
            for (int j = 0; j < SEG; ++j) {
                fa[j] = *reinterpret_cast<const uint4 *>(pa + j * 64);
                fc[j] = *reinterpret_cast<const uint4 *>(pa + 8 * ROWB + j * 64);
            }
        }
        const int rel_stage = cs;
        if (++cs == kP1Stages) {
            cs = 0;
            cph ^= 1u;
        }
        for (int qb = 0; qb < GW; qb += kQB) {
            if (!one_block) {
                csync();  // the previous block's tile and queries are no longer read
                load_queries(qb);
            }
            csync();      // queries in place; the previous chunk's tile is no longer read
#pragma unroll
            for (int nb = 0; nb < kQB / 8; ++nb) {
                float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
                const uint8_t *pq = Qs + (nb * 8 + gq) * ROWB + tig * 16;
#pragma unroll
                for (int j = 0; j < SEG; ++j) {
                    const uint4 qv = *reinterpret_cast<const uint4 *>(pq + j * 64);
                    mma_16x8x16<T>(c0, fa[j].x, fc[j].x, fa[j].y, fc[j].y, qv.x, qv.y);
                    mma_16x8x16<T>(c1, fa[j].z, fc[j].z, fa[j].w, fc[j].w, qv.z, qv.w);
                }
                // rows gq, gq+8 of the warp's positions; query rows nb*8 + tig*2, +1
                const int pos = warp * 16 + gq;
                const int qr = nb * 8 + tig * 2;
                lt[qr * LT + pos] = (c0[0] + c1[0]) * p.scale;
                lt[(qr + 1) * LT + pos] = (c0[1] + c1[1]) * p.scale;
                lt[qr * LT + pos + 8] = (c0[2] + c1[2]) * p.scale;
                lt[(qr + 1) * LT + pos + 8] = (c0[3] + c1[3]) * p.scale;
            }
            if (qb == 0) {
                // The stage goes back once the fragments have been used, not merely requested:
                // an arrival issued right behind the shared-memory loads can be seen by the
                // producer before their data has been read (measured: wrong logits).
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[rel_stage]);
            }
            csync();
            // warp w: query rows 4w .. 4w+3 of the block; lane: positions lane + 32 i
#pragma unroll
            for (int jr = 0; jr < 4; ++jr) {
                const int gw = qb + warp * 4 + jr;
                if (gw >= GW) continue;  // uniform per warp
                const int tau = T_len - W + (gw % W);  // the query's own position: keys 0..tau
                float m = -INFINITY;
                float lg[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int t = t0 + lane + 32 * i;
                    lg[i] = (t < T_len && t <= tau) ? lt[(warp * 4 + jr) * LT + lane + 32 * i] : -INFINITY;
                    if (t < T_len) logits[(size_t)gw * T_len + t] = lg[i];
                    m = fmaxf(m, lg[i]);
                }
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
                float sum = 0.f;
                if (m > -INFINITY) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) sum += expf(lg[i] - m);
                }
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
                if (lane == 0) partial[(size_t)gw * n_chunks + chunk] = make_float2(m, sum);
            }
        }
    }
}

template <int D>
size_t logits_mma_smem_bytes() {
    return (size_t)(kP1Stages * kPrefillChunk + kQB) * D * 2 + (size_t)kQB * (kPrefillChunk + 4) * 4 +
           (size_t)(2 * kP1Stages) * 8 + 64;
}

// P1b: one thread per (unit, query row): fold the chunk partials.
__global__ void prefill_rowstat_kernel(const PrefillParams p, int n_chunks) {
    const int GW = p.G * p.W;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= p.units * GW) return;
    const float2 *part = reinterpret_cast<const float2 *>(p.ws + p.wl.partial) + (size_t)idx * n_chunks;
    float m = -INFINITY;
    for (int c = 0; c < n_chunks; ++c) m = fmaxf(m, part[c].x);
    float z = 0.f;
    for (int c = 0; c < n_chunks; ++c) {
        const float2 v = part[c];
        if (v.x > -INFINITY) z += v.y * expf(v.x - m);
    }
    const int wq = idx % p.W;
    // weight of query position tau = T-W+wq in Eq. (score) unrolled, and the group mean
    const double coef = pow(static_cast<double>(p.lambda), static_cast<double>(p.W - 1 - wq)) /
                        static_cast<double>(p.G);
    reinterpret_cast<float2 *>(p.ws + p.wl.rowstat)[idx] =
        make_float2(m, static_cast<float>(coef / static_cast<double>(z)));
}

// P1c: one thread per (unit, position).
__global__ void prefill_scores_kernel(const PrefillParams p) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int ul = blockIdx.y;
    if (t >= p.T) return;
    const int GW = p.G * p.W;
    const float *logits = reinterpret_cast<const float *>(p.ws + p.wl.logits) + (size_t)ul * GW * p.T;
    const float2 *rs = reinterpret_cast<const float2 *>(p.ws + p.wl.rowstat) + (size_t)ul * GW;
    float s = 0.f;
    for (int gw = 0; gw < GW; ++gw) {
        const float2 st = __ldg(rs + gw);
        s = fmaf(expf(logits[(size_t)gw * p.T + t] - st.x), st.y, s);
    }
    reinterpret_cast<float *>(p.ws + p.wl.scores)[(size_t)ul * p.T + t] = s;
}

// ---------------------------------------------------------------------------
// P2 + P3: one CTA per unit.  Radix select (8 bits per pass, most significant
// first) of the n_ev-th smallest (score, position) key among the candidates,
// then two ordered compactions.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) prefill_select_kernel(const PrefillParams p,
                                                              const float *scores) {
    __shared__ uint32_t hist[256];
    __shared__ uint64_t s_prefix;
    __shared__ uint32_t s_k;
    __shared__ uint32_t wsum_e[32], wsum_k[32];
    __shared__ uint32_t base_e, base_k;

    const int ul = blockIdx.x;
    const UnitDesc d = p.desc[ul];
    const int T_len = p.T;
    const int n_prox = min(T_len, d.Bp);
    const int n_cand = T_len - n_prox;
    const int n_ev = max(0, n_cand - d.Bc);
    const float *s = scores + (size_t)ul * T_len;
    uint8_t *flags = p.ws + p.wl.flags + (size_t)ul * T_len;
    int32_t *evl = reinterpret_cast<int32_t *>(p.ws + p.wl.evict_list) + (size_t)ul * T_len;
    int32_t *kpl = reinterpret_cast<int32_t *>(p.ws + p.wl.kept_list) + (size_t)ul * T_len;
    const int tid = threadIdx.x;

    auto key_of = [&](int t) -> uint64_t {
        return (static_cast<uint64_t>(score_order_bits(s[t])) << 32) | static_cast<uint32_t>(t);
    };

    uint64_t thr = 0;
    if (n_ev > 0) {
        if (tid == 0) {
            s_prefix = 0;
            s_k = static_cast<uint32_t>(n_ev);
        }
        for (int pass = 7; pass >= 0; --pass) {
            const int shift = pass * 8;
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            const uint64_t prefix = s_prefix;
            for (int t = tid; t < n_cand; t += blockDim.x) {
                const uint64_t key = key_of(t);
                const bool match = (pass == 7) || ((key >> (shift + 8)) == (prefix >> (shift + 8)));
                if (match) atomicAdd(&hist[(key >> shift) & 255u], 1u);
            }
            __syncthreads();
            if (tid == 0) {
                uint32_t k = s_k, cum = 0;
                int dg = 0;
                for (; dg < 256; ++dg) {
                    if (cum + hist[dg] >= k) break;
                    cum += hist[dg];
                }
                s_k = k - cum;
                s_prefix = prefix | (static_cast<uint64_t>(dg) << shift);
            }
            __syncthreads();
        }
        thr = s_prefix;
    }

    if (tid == 0) {
        base_e = 0;
        base_k = 0;
    }
    __syncthreads();
    const int lane = tid & 31, warp = tid >> 5;
    for (int t0 = 0; t0 < T_len; t0 += blockDim.x) {
        const int t = t0 + tid;
        const bool in = t < T_len;
        const bool ev = in && n_ev > 0 && t < n_cand && key_of(t) <= thr;
        if (in && s[t] != s[t]) dev_set_status(p.status, DEV_ERR_CHECK, d.unit, 5);  // NaN score
        const bool kp = in && !ev;
        if (in) flags[t] = ev ? 1 : 0;
        const uint32_t be = __ballot_sync(0xffffffffu, ev);
        const uint32_t bk = __ballot_sync(0xffffffffu, kp);
        if (lane == 0) {
            wsum_e[warp] = __popc(be);
            wsum_k[warp] = __popc(bk);
        }
        __syncthreads();
        uint32_t oe = base_e, ok = base_k;
        for (int wv = 0; wv < warp; ++wv) {
            oe += wsum_e[wv];
            ok += wsum_k[wv];
        }
        const uint32_t lt = (1u << lane) - 1u;
        if (ev) evl[oe + __popc(be & lt)] = t;
        if (kp) kpl[ok + __popc(bk & lt)] = t;
        __syncthreads();
        if (tid == 0) {
            uint32_t te = 0, tk = 0;
            for (int wv = 0; wv < (int)(blockDim.x >> 5); ++wv) {
                te += wsum_e[wv];
                tk += wsum_k[wv];
            }
            base_e += te;
            base_k += tk;
        }
        __syncthreads();
    }
    if (tid == 0) {
        int32_t *cnt = reinterpret_cast<int32_t *>(p.ws + p.wl.counts) + ul * 4;
        cnt[0] = static_cast<int32_t>(base_e);
        cnt[1] = static_cast<int32_t>(base_k);
        if (static_cast<int32_t>(base_e) != n_ev) dev_set_status(p.status, DEV_ERR_CHECK, d.unit, 3);
    }
    if (p.dbg_evicted) {
        __syncthreads();
        for (int t = tid; t < T_len; t += blockDim.x) p.dbg_evicted[(size_t)ul * T_len + t] = flags[t];
    }
    if (p.dbg_scores) {
        for (int t = tid; t < T_len; t += blockDim.x) p.dbg_scores[(size_t)ul * T_len + t] = s[t];
    }
}

// ---------------------------------------------------------------------------
// P4: one CTA per unit walks the evicted tokens in ascending position.  The B_r
// residual rows live in shared memory as fp32; evicted rows arrive through a small
// cp.async ring, several tokens ahead of the merge that needs them.
// ---------------------------------------------------------------------------
constexpr int kMergeWarps = 8;
constexpr int kMergePF = 8;     // ring slots
constexpr int kMergeIB = 512;   // evicted positions staged in shared memory at a time

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <typename T, int D>
__global__ void __launch_bounds__(kMergeWarps * 32) prefill_merge_kernel(const PrefillParams p) {
    using E = Elem<T>;
    constexpr int ROWB = D * (int)sizeof(T);
    constexpr int CPR = ROWB / 16;  // 16-byte chunks per row
    constexpr int EPT = D / 32;     // elements per lane
    static_assert(2 * CPR <= kMergeWarps * 32, "one cp.async per thread covers a K and a V row");
    extern __shared__ __align__(16) uint8_t smraw[];

    const int ul = blockIdx.x;
    const UnitDesc d = p.desc[ul];
    const int Br = d.Br;
    const int T_len = p.T;
    const int n_ev = reinterpret_cast<const int32_t *>(p.ws + p.wl.counts)[ul * 4];
    const int32_t *evl = reinterpret_cast<const int32_t *>(p.ws + p.wl.evict_list) + (size_t)ul * T_len;
    int32_t *targets = p.dbg_targets ? p.dbg_targets + (size_t)ul * T_len : nullptr;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (Br == 0) {
        if (targets)
            for (int i = tid; i < n_ev; i += blockDim.x) targets[i] = -1;  // dropped (Sec. 3.2)
        return;
    }
    const int br_pad = (Br + 3) & ~3;
    float *Kr_s = reinterpret_cast<float *>(smraw);
    float *Vr_s = Kr_s + (size_t)Br * D;
    float *dots_s = Vr_s + (size_t)Br * D;
    uint32_t *w_s = reinterpret_cast<uint32_t *>(dots_s + br_pad);
    int32_t *idx_s = reinterpret_cast<int32_t *>(w_s + br_pad);         // [kMergeIB + kMergePF]
    uint8_t *ring = reinterpret_cast<uint8_t *>(idx_s + kMergeIB + kMergePF);  // [PF][2][ROWB]

    const uint8_t *Kg = static_cast<const uint8_t *>(p.K) + (size_t)ul * T_len * ROWB;
    const uint8_t *Vg = static_cast<const uint8_t *>(p.V) + (size_t)ul * T_len * ROWB;

    // idx_s[j] = evl[i0 + j] for the current block of evicted tokens starting at i0
    int i0 = 0;
    auto stage_indices = [&](int start) {
        for (int j = tid; j < kMergeIB + kMergePF; j += blockDim.x)
            idx_s[j] = (start + j < n_ev) ? evl[start + j] : 0;
    };
    auto issue = [&](int i) {  // fetch evicted token i's rows into ring slot i % PF
        if (i < n_ev && tid < 2 * CPR) {
            const int which = tid / CPR, c = tid % CPR;
            const int t = idx_s[i - i0];
            const uint8_t *src = (which ? Vg : Kg) + (size_t)t * ROWB + c * 16;
            cp_async16(ring + ((size_t)(i % kMergePF) * 2 + which) * ROWB + c * 16, src);
        }
        cp_async_commit();
    };

    stage_indices(0);
    __syncthreads();
    for (int i = 0; i < kMergePF - 1; ++i) issue(i);

    for (int i = 0; i < n_ev; ++i) {
        if (i - i0 == kMergeIB) {  // next block of positions (every thread is past iteration i-1)
            i0 = i;
            stage_indices(i0);
            __syncthreads();
        }
        issue(i + kMergePF - 1);
        cp_async_wait<kMergePF - 1>();
        __syncthreads();  // token i's rows are in the ring for everyone
        const T *kc_row = reinterpret_cast<const T *>(ring + ((size_t)(i % kMergePF) * 2 + 0) * ROWB);
        const T *vc_row = reinterpret_cast<const T *>(ring + ((size_t)(i % kMergePF) * 2 + 1) * ROWB);
        if (i < Br) {
            // Alg. 1 l.12-13: free slot
            for (int k = tid; k < D; k += blockDim.x) {
                Kr_s[(size_t)i * D + k] = E::to_float(kc_row[k]);
                Vr_s[(size_t)i * D + k] = E::to_float(vc_row[k]);
            }
            if (tid == 0) {
                w_s[i] = 1;
                if (targets) targets[i] = -2;
            }
        } else {
            float kc[EPT];
            float nt2 = 0.f;  // |k_t|^2, for the cosine form
#pragma unroll
            for (int e = 0; e < EPT; ++e) {
                kc[e] = E::to_float(kc_row[lane * EPT + e]);
                nt2 = fmaf(kc[e], kc[e], nt2);
            }
            if (p.cosine) {
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) nt2 += __shfl_xor_sync(0xffffffffu, nt2, off);
            }
            for (int r = warp; r < Br; r += kMergeWarps) {  // Eq. (hatr)
                const float *kr = Kr_s + (size_t)r * D + lane * EPT;
                float acc = 0.f, nr2 = 0.f;
#pragma unroll
                for (int e = 0; e < EPT; ++e) {
                    acc = fmaf(kr[e], kc[e], acc);
                    nr2 = fmaf(kr[e], kr[e], nr2);
                }
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
                if (p.cosine) {
#pragma unroll
                    for (int off = 16; off >= 1; off >>= 1) nr2 += __shfl_xor_sync(0xffffffffu, nr2, off);
                    const float nn = sqrtf(nr2) * sqrtf(nt2);
                    acc = nn > 0.f ? acc / nn : 0.f;
                }
                if (lane == 0) dots_s[r] = acc;
            }
            __syncthreads();
            float bd = -INFINITY;
            int br = 0x7fffffff;
            for (int r = lane; r < Br; r += 32) {
                const float dv = dots_s[r];
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
            if (warp == br % kMergeWarps) {  // Eq. (kvr)
                const float wr = static_cast<float>(w_s[br]);
                float *kr = Kr_s + (size_t)br * D + lane * EPT;
                float *vr = Vr_s + (size_t)br * D + lane * EPT;
#pragma unroll
                for (int e = 0; e < EPT; ++e) {
                    kr[e] = fmaf(wr, kr[e], kc[e]) / (wr + 1.0f);
                    vr[e] = fmaf(wr, vr[e], E::to_float(vc_row[lane * EPT + e])) / (wr + 1.0f);
                }
                __syncwarp();
                if (lane == 0) {
                    w_s[br] += 1u;
                    if (targets) targets[i] = br;
                }
            }
        }
        __syncthreads();  // rows updated; ring slot i % PF may be refilled
    }
    cp_async_wait<0>();

    const int n_res = min(Br, n_ev);
    float *Kr_g = reinterpret_cast<float *>(p.base + d.kr_off);
    float *Vr_g = reinterpret_cast<float *>(p.base + d.vr_off);
    uint32_t *w_g = reinterpret_cast<uint32_t *>(p.base + d.w_off);
    for (int k = tid; k < n_res * D; k += blockDim.x) {
        Kr_g[k] = Kr_s[k];
        Vr_g[k] = Vr_s[k];
    }
    for (int k = tid; k < n_res; k += blockDim.x) w_g[k] = w_s[k];
}

// ---------------------------------------------------------------------------
// P4, row-per-warp form (B_r <= 32 * RT): one CTA of 32 warps per unit.  Warp r keeps merged
// key and value rows r, r + 32, .. in registers, D/32 elements per lane, so a dot product is
// D/32 FMAs and five shuffles, and an update touches registers only.  Per evicted token: every
// warp dots its rows with the token's key and posts its best (order-preserving key, slot) to
// shared memory; one barrier; every warp reads the 32 posts with one load per lane and settles
// the argmax with two integer warp reductions (lowest slot wins ties); the owning warp applies
// Eq. (kvr).  A single warp issues roughly one instruction every four cycles, so the chain's
// speed is the number of instructions on one warp's critical path: about 60 here.
// Evicted rows arrive through a cp.async ring several tokens ahead.
// ---------------------------------------------------------------------------
constexpr int kRowMergeThreads = 1024;
constexpr int kRowMergePF = 10;  // ring slots; a slot is refilled two tokens after its use
constexpr int kRowMergeIdx = (kMergeIB + kRowMergePF + 3) & ~3;  // staged positions, padded so
                                                                 // the ring after them stays
                                                                 // 16-byte aligned for cp.async

__device__ __forceinline__ uint32_t order_key(float f) {  // a < b  <=>  key(a) < key(b); key > 0
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <typename T, int D, int RT>
__global__ void __launch_bounds__(kRowMergeThreads) prefill_merge_rows_kernel(const PrefillParams p) {
    using E = Elem<T>;
    constexpr int ROWB = D * (int)sizeof(T);
    constexpr int CPR = ROWB / 16;   // 16-byte chunks per row
    constexpr int EPT = D / 32;      // elements of a row per lane
    constexpr int PF = kRowMergePF;
    static_assert(2 * CPR <= kRowMergeThreads, "one cp.async per thread covers a K and a V row");
    static_assert((64 * 4 + kRowMergeIdx * 4) % 16 == 0, "the ring starts on a 16-byte boundary");
    extern __shared__ __align__(16) uint8_t smraw[];

    const int ul = blockIdx.x;
    const UnitDesc d = p.desc[ul];
    const int Br = d.Br;
    const int T_len = p.T;
    const int n_ev = reinterpret_cast<const int32_t *>(p.ws + p.wl.counts)[ul * 4];
    const int32_t *evl = reinterpret_cast<const int32_t *>(p.ws + p.wl.evict_list) + (size_t)ul * T_len;
    int32_t *targets = p.dbg_targets ? p.dbg_targets + (size_t)ul * T_len : nullptr;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (Br == 0) {
        if (targets)
            for (int i = tid; i < n_ev; i += blockDim.x) targets[i] = -1;  // dropped (Sec. 3.2)
        return;
    }
    uint32_t *best_k = reinterpret_cast<uint32_t *>(smraw);                  // [2][32] warps' best keys
    int32_t *best_r = reinterpret_cast<int32_t *>(best_k + 64);              // [2][32] and their slots
    int32_t *idx_s = best_r + 64;                                            // [kRowMergeIdx]
    uint8_t *ring = reinterpret_cast<uint8_t *>(idx_s + kRowMergeIdx);       // [PF][2][ROWB]

    const uint8_t *Kg = static_cast<const uint8_t *>(p.K) + (size_t)ul * T_len * ROWB;
    const uint8_t *Vg = static_cast<const uint8_t *>(p.V) + (size_t)ul * T_len * ROWB;

    float kr[RT][EPT], vr[RT][EPT];  // this lane's elements of the warp's merged rows
    float wr[RT];                    // their fusion counts
#pragma unroll
    for (int j = 0; j < RT; ++j) {
        wr[j] = 0.f;
#pragma unroll
        for (int e = 0; e < EPT; ++e) kr[j][e] = vr[j][e] = 0.f;
    }

    int i0 = 0;  // idx_s[j] = evl[i0 + j]
    auto stage_indices = [&](int start) {
        for (int j = tid; j < kRowMergeIdx; j += blockDim.x)
            idx_s[j] = (start + j < n_ev) ? evl[start + j] : 0;
    };
    auto issue = [&](int i) {  // fetch evicted token i's rows into ring slot i % PF
        if (i < n_ev && tid < 2 * CPR) {
            const int which = tid / CPR, c = tid % CPR;
            const int t = idx_s[i - i0];
            const uint8_t *src = (which ? Vg : Kg) + (size_t)t * ROWB + c * 16;
            cp_async16(ring + ((size_t)(i % PF) * 2 + which) * ROWB + c * 16, src);
        }
        cp_async_commit();
    };
    auto load_own = [&](const uint8_t *rowp, float (&f)[EPT]) {
        const T *src = reinterpret_cast<const T *>(rowp) + lane * EPT;
#pragma unroll
        for (int e = 0; e < EPT; ++e) f[e] = E::to_float(src[e]);
    };

    stage_indices(0);
    __syncthreads();
    for (int i = 0; i < PF - 2; ++i) issue(i);  // tokens 0 .. PF-3 in flight
    cp_async_wait<PF - 3>();                    // token 0 has landed
    __syncthreads();

    for (int i = 0; i < n_ev; ++i) {
        // ring slot of token i-2 is free (its last readers passed the barrier of token i-1)
        issue(i + PF - 2);
        const uint8_t *kc_row = ring + ((size_t)(i % PF) * 2 + 0) * ROWB;
        const uint8_t *vc_row = ring + ((size_t)(i % PF) * 2 + 1) * ROWB;
        const int par = (i & 1) * 32;
        float kc[EPT];
        load_own(kc_row, kc);
        int target = -1;
        if (i < Br) {
            target = i;  // Alg. 1: a free residual slot takes the token as it is
        } else {
            // Eq. (hatr): raw dot products; within the warp ties go to the lower slot
            float dot[RT];
#pragma unroll
            for (int j = 0; j < RT; ++j) {
                float a = 0.f;
#pragma unroll
                for (int e = 0; e < EPT; ++e) a = fmaf(kr[j][e], kc[e], a);
                dot[j] = a;
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1)
#pragma unroll
                for (int j = 0; j < RT; ++j) dot[j] += __shfl_xor_sync(0xffffffffu, dot[j], off);
            float bv = 0.f;
            int br = 0x7fffffff;
#pragma unroll
            for (int j = 0; j < RT; ++j) {
                const int r = warp + 32 * j;
                if (r < Br && (br == 0x7fffffff || dot[j] > bv)) {
                    bv = dot[j];
                    br = r;
                }
            }
            if (lane == 0) {
                best_k[par + warp] = br == 0x7fffffff ? 0u : order_key(bv);
                best_r[par + warp] = br;
            }
        }
        // token i+1 must have landed before the barrier that publishes it
        cp_async_wait<PF - 3>();
        __syncthreads();
        if (target < 0) {
            const uint32_t key = best_k[par + lane];
            const uint32_t mx = __reduce_max_sync(0xffffffffu, key);
            const int r = key == mx ? best_r[par + lane] : 0x7fffffff;
            target = __reduce_min_sync(0xffffffffu, r);
        }
        // Eq. (kvr) on the chosen row, by its warp
        if ((target & 31) == warp) {
#pragma unroll
            for (int j = 0; j < RT; ++j) {
                if (warp + 32 * j == target) {
                    const float w = wr[j];
                    // one correctly rounded reciprocal instead of divisions on the critical path
                    const float rdn = __frcp_rn(w + 1.0f);
                    float vc[EPT];
                    load_own(vc_row, vc);
#pragma unroll
                    for (int e = 0; e < EPT; ++e) {
                        kr[j][e] = (w == 0.f) ? kc[e] : fmaf(w, kr[j][e], kc[e]) * rdn;
                        vr[j][e] = (w == 0.f) ? vc[e] : fmaf(w, vr[j][e], vc[e]) * rdn;
                    }
                    wr[j] = w + 1.0f;
                    if (lane == 0 && targets) targets[i] = (i < Br) ? -2 : target;
                }
            }
        }
        if (i + 1 - i0 == kMergeIB && i + 1 < n_ev) {
            // next block of positions; tokens up to i + PF - 2 were issued from the old block,
            // whose tail covers them
            __syncthreads();
            i0 = i + 1;
            stage_indices(i0);
            __syncthreads();
        }
    }
    cp_async_wait<0>();

    const int n_res = min(Br, n_ev);
    float *Kr_g = reinterpret_cast<float *>(p.base + d.kr_off);
    float *Vr_g = reinterpret_cast<float *>(p.base + d.vr_off);
    uint32_t *w_g = reinterpret_cast<uint32_t *>(p.base + d.w_off);
#pragma unroll
    for (int j = 0; j < RT; ++j) {
        const int r = warp + 32 * j;
        if (r < n_res) {
#pragma unroll
            for (int e = 0; e < EPT; ++e) {
                Kr_g[(size_t)r * D + lane * EPT + e] = kr[j][e];
                Vr_g[(size_t)r * D + lane * EPT + e] = vr[j][e];
            }
            if (lane == 0) w_g[r] = static_cast<uint32_t>(wr[j]);
        }
    }
}

template <typename T, int D>
size_t merge_rows_smem_bytes() {
    return (size_t)128 * 4 + (size_t)kRowMergeIdx * 4 + (size_t)kRowMergePF * 2 * D * sizeof(T);
}

// ---------------------------------------------------------------------------
// P4, one-warp form (B_r <= 32), for layers with more units than the GPU can hold CTAs of
// the row-per-warp form: a single warp walks a unit's chain, so a merge costs no block barrier
// and every unit of the layer runs at once.  Lane r owns merged key r (a shared-memory row padded to D + 1 floats,
// which makes the lanes' row-wise reads conflict-free); the token's key is widened to fp32 once,
// cooperatively, and broadcast-read by every lane for its dot product; the argmax is one
// integer warp reduction on order-preserving keys plus a ballot (lowest slot wins ties); the
// chosen row and its value row are updated cooperatively, D/32 elements per lane.
// ---------------------------------------------------------------------------
constexpr int kWarpMergePF = 8;     // ring slots
constexpr int kWarpMergeIB = 120;   // evicted positions staged at a time (IB + PF: multiple of 4)

template <typename T, int D>
__global__ void __launch_bounds__(32) prefill_merge_warp_kernel(const PrefillParams p) {
    using E = Elem<T>;
    constexpr int ROWB = D * (int)sizeof(T);
    constexpr int CPR = ROWB / 16;
    constexpr int EPTL = D / 32;  // elements of a row per lane in the cooperative steps
    constexpr int LD = D + 1;     // padded key row
    constexpr int PF = kWarpMergePF, IB = kWarpMergeIB;
    static_assert((32 * LD * 4) % 16 == 0 && ((IB + PF) * 4) % 16 == 0, "16-byte aligned ring");
    extern __shared__ __align__(16) uint8_t smraw[];

    const int ul = blockIdx.x;
    const UnitDesc d = p.desc[ul];
    const int Br = d.Br;
    const int T_len = p.T;
    const int n_ev = reinterpret_cast<const int32_t *>(p.ws + p.wl.counts)[ul * 4];
    const int32_t *evl = reinterpret_cast<const int32_t *>(p.ws + p.wl.evict_list) + (size_t)ul * T_len;
    int32_t *targets = p.dbg_targets ? p.dbg_targets + (size_t)ul * T_len : nullptr;
    const int lane = threadIdx.x;

    if (Br == 0) {
        if (targets)
            for (int i = lane; i < n_ev; i += 32) targets[i] = -1;  // dropped (Sec. 3.2)
        return;
    }
    float *Kr_s = reinterpret_cast<float *>(smraw);               // [32][LD]
    float *Vr_s = Kr_s + 32 * LD;                                 // [32][D]
    float *kcf = Vr_s + 32 * D;                                   // [D] the token's key, fp32
    int32_t *idx_s = reinterpret_cast<int32_t *>(kcf + D);        // [IB + PF]
    uint8_t *ring = reinterpret_cast<uint8_t *>(idx_s + IB + PF); // [PF][2][ROWB]

    const uint8_t *Kg = static_cast<const uint8_t *>(p.K) + (size_t)ul * T_len * ROWB;
    const uint8_t *Vg = static_cast<const uint8_t *>(p.V) + (size_t)ul * T_len * ROWB;

    float wr = 0.f;  // fusion count of slot `lane`
    int i0 = 0;
    auto stage_indices = [&](int start) {
        for (int j = lane; j < IB + PF; j += 32) idx_s[j] = (start + j < n_ev) ? evl[start + j] : 0;
    };
    auto issue = [&](int i) {
        if (i < n_ev) {
            const int t = idx_s[i - i0];
            for (int c = lane; c < 2 * CPR; c += 32) {
                const int which = c / CPR, cc = c % CPR;
                cp_async16(ring + ((size_t)(i % PF) * 2 + which) * ROWB + cc * 16,
                           (which ? Vg : Kg) + (size_t)t * ROWB + cc * 16);
            }
        }
        cp_async_commit();
    };

    stage_indices(0);
    __syncwarp();
    for (int i = 0; i < PF - 1; ++i) issue(i);

    for (int i = 0; i < n_ev; ++i) {
        if (i - i0 == IB) {  // next block of positions
            __syncwarp();
            i0 = i;
            stage_indices(i0);
            __syncwarp();
        }
        issue(i + PF - 1);  // refills the slot of token i-1, which the warp is done with
        cp_async_wait<PF - 1>();
        __syncwarp();  // token i's rows are in the ring for every lane
        const T *kc_row = reinterpret_cast<const T *>(ring + ((size_t)(i % PF) * 2 + 0) * ROWB);
        const T *vc_row = reinterpret_cast<const T *>(ring + ((size_t)(i % PF) * 2 + 1) * ROWB);
        float kc[EPTL], vc[EPTL];
#pragma unroll
        for (int e = 0; e < EPTL; ++e) {
            kc[e] = E::to_float(kc_row[lane * EPTL + e]);
            vc[e] = E::to_float(vc_row[lane * EPTL + e]);
            kcf[lane * EPTL + e] = kc[e];
        }
        __syncwarp();
        int target;
        if (i < Br) {
            target = i;  // Alg. 1: a free residual slot takes the token as it is
        } else {
            // Eq. (hatr): lane r's dot product of merged key r with the token's key
            const float *kr = Kr_s + lane * LD;
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 8
            for (int k = 0; k < D; k += 4) {
                const float4 c4 = *reinterpret_cast<const float4 *>(kcf + k);
                a0 = fmaf(kr[k], c4.x, a0);
                a1 = fmaf(kr[k + 1], c4.y, a1);
                a2 = fmaf(kr[k + 2], c4.z, a2);
                a3 = fmaf(kr[k + 3], c4.w, a3);
            }
            const float dot = (a0 + a1) + (a2 + a3);
            const uint32_t key = lane < Br ? order_key(dot) : 0u;
            const uint32_t best = __reduce_max_sync(0xffffffffu, key);
            target = __ffs(__ballot_sync(0xffffffffu, key == best && lane < Br)) - 1;
        }
        // Eq. (kvr) on the chosen row, D/32 elements per lane
        const float w = __shfl_sync(0xffffffffu, wr, target);
        const float rdn = __frcp_rn(w + 1.0f);
        float *krow = Kr_s + target * LD + lane * EPTL;
        float *vrow = Vr_s + target * D + lane * EPTL;
#pragma unroll
        for (int e = 0; e < EPTL; ++e) {
            krow[e] = (w == 0.f) ? kc[e] : fmaf(w, krow[e], kc[e]) * rdn;
            vrow[e] = (w == 0.f) ? vc[e] : fmaf(w, vrow[e], vc[e]) * rdn;
        }
        if (lane == target) wr = w + 1.0f;
        if (lane == 0 && targets) targets[i] = (i < Br) ? -2 : target;
        __syncwarp();  // the updated row is in place before the next token's dot products
    }
    cp_async_wait<0>();
    __syncwarp();

    const int n_res = min(Br, n_ev);
    float *Kr_g = reinterpret_cast<float *>(p.base + d.kr_off);
    float *Vr_g = reinterpret_cast<float *>(p.base + d.vr_off);
    uint32_t *w_g = reinterpret_cast<uint32_t *>(p.base + d.w_off);
    for (int k = lane; k < n_res * D; k += 32) {
        Kr_g[k] = Kr_s[(k / D) * LD + (k % D)];
        Vr_g[k] = Vr_s[k];
    }
    if (lane < n_res) w_g[lane] = static_cast<uint32_t>(wr);
}

template <typename T, int D>
size_t merge_warp_smem_bytes() {
    return (size_t)32 * (D + 1) * 4 + (size_t)32 * D * 4 + (size_t)D * 4 +
           (size_t)(kWarpMergeIB + kWarpMergePF) * 4 + (size_t)kWarpMergePF * 2 * D * sizeof(T);
}

// ---------------------------------------------------------------------------
// P4, blocked form (16-bit storage, B_r <= 32): the chain is still walked token by token, but
// what a token needs from the merged keys is no longer a D-long dot product per slot.  For a
// block of 64 evicted tokens the dot products with the merged keys as they stood at the start
// of the block (D0 = K_blk Kr^T) and the tokens' own Gram matrix (Gm = K_blk K_blk^T) are
// formed at once on the tensor cores.  Because a merged key is the mean of its constituents,
//     k_r . k_t  =  ( w0_r * D0[t][r] + sum over block tokens u already merged into r of Gm[t][u] ) / w_r
// so one warp walks the block keeping that numerator per (token, slot): per token one shared
// load per lane, a multiply by 1/w_r, an integer warp reduction for the argmax (lowest slot wins
// ties), and the Gram row of the token added to the chosen slot's numerators of the later
// tokens.  After the block, every slot's key and value are rebuilt from its old mean and the
// sum of the tokens it took.  The arithmetic is that of Eq. (hatr)/(kvr) reassociated.
// The merged keys enter the tensor cores as three 16-bit pieces (hi + mid + lo = the fp32
// value to its last bit), so D0 is an fp32-accumulated product of exact operands.
// ---------------------------------------------------------------------------
constexpr int kBlkTokens = 64;
constexpr int kBlkGS = kBlkTokens + 4;  // row stride of the Gram matrix

template <int D, int NS>
struct BlkSmem {
    static constexpr int ROWB = D * 2;
    static constexpr size_t tokK = 0;                                        // [2][64][ROWB]
    static constexpr size_t tokV = tokK + 2 * kBlkTokens * ROWB;             // [2][64][ROWB]
    static constexpr size_t krm = tokV + 2 * kBlkTokens * ROWB;              // [NS][D] fp32
    static constexpr size_t vrm = krm + NS * D * 4;                          // [NS][D] fp32
    static constexpr size_t krs = vrm + NS * D * 4;                          // [3][NS][D] 16-bit
    static constexpr size_t num = krs + 3 * NS * ROWB;                       // [64][NS + 1] fp32
    static constexpr size_t gm = num + kBlkTokens * (NS + 1) * 4;            // [64][68] fp32
    static constexpr size_t tgt = gm + kBlkTokens * kBlkGS * 4;              // [64] int
    static constexpr size_t wc = tgt + kBlkTokens * 4;                       // [NS] fp32 counts
    static constexpr size_t total = wc + NS * 4;
};

template <typename T, int D, int NS>
__global__ void __launch_bounds__(1024) prefill_merge_blocked_kernel(const PrefillParams p) {
    using E = Elem<T>;
    using SM = BlkSmem<D, NS>;
    constexpr int NS1 = NS + 1;   // row stride of the numerator table (bank-conflict free)
    constexpr int SPL = NS / 32;  // merged slots a lane of the chain warp watches
    constexpr int NTD = NS / 8;   // 8-slot column tiles of the numerator table
    static_assert(sizeof(T) == 2, "16-bit storage");
    constexpr int ROWB = D * 2;
    constexpr int CPR = ROWB / 16;
    constexpr int SEG = ROWB / 64;
    constexpr int EPT = D / 32;
    constexpr int NB = kBlkTokens;
    extern __shared__ __align__(16) uint8_t smraw[];

    const int ul = blockIdx.x;
    const UnitDesc d = p.desc[ul];
    const int Br = d.Br;
    const int T_len = p.T;
    const int n_ev = reinterpret_cast<const int32_t *>(p.ws + p.wl.counts)[ul * 4];
    const int32_t *evl = reinterpret_cast<const int32_t *>(p.ws + p.wl.evict_list) + (size_t)ul * T_len;
    int32_t *targets = p.dbg_targets ? p.dbg_targets + (size_t)ul * T_len : nullptr;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_warps = blockDim.x >> 5;
    const int gq = lane >> 2, tig = lane & 3;

    if (Br == 0) {
        if (targets)
            for (int i = tid; i < n_ev; i += blockDim.x) targets[i] = -1;  // dropped (Sec. 3.2)
        return;
    }
    uint8_t *tokK = smraw + SM::tokK, *tokV = smraw + SM::tokV;
    float *KrM = reinterpret_cast<float *>(smraw + SM::krm);
    float *VrM = reinterpret_cast<float *>(smraw + SM::vrm);
    uint8_t *KrS = smraw + SM::krs;
    float *Num = reinterpret_cast<float *>(smraw + SM::num);
    float *Gm = reinterpret_cast<float *>(smraw + SM::gm);
    int32_t *tgt = reinterpret_cast<int32_t *>(smraw + SM::tgt);
    float *wc = reinterpret_cast<float *>(smraw + SM::wc);

    const uint8_t *Kg = static_cast<const uint8_t *>(p.K) + (size_t)ul * T_len * ROWB;
    const uint8_t *Vg = static_cast<const uint8_t *>(p.V) + (size_t)ul * T_len * ROWB;

    // element e of merged key row r as three 16-bit pieces for the tensor cores
    auto write_split = [&](int r, int e, float x) {
        T *s0 = reinterpret_cast<T *>(KrS) + (size_t)r * D + e;
        const T h = E::from_float(x);
        const float r1 = x - E::to_float(h);
        const T m = E::from_float(r1);
        const T l = E::from_float(r1 - E::to_float(m));
        s0[0] = h;
        s0[NS * D] = m;
        s0[2 * NS * D] = l;
    };

    // ---- fill: the first B_r evicted tokens take the free slots as they are (Alg. 1) ----
    const int n_fill = min(Br, n_ev);
    for (int k = tid; k < NS * D; k += blockDim.x) {
        const int r = k / D, e = k % D;
        float kv = 0.f, vv = 0.f;
        if (r < n_fill) {
            const int t = evl[r];
            kv = E::to_float(reinterpret_cast<const T *>(Kg + (size_t)t * ROWB)[e]);
            vv = E::to_float(reinterpret_cast<const T *>(Vg + (size_t)t * ROWB)[e]);
        }
        KrM[k] = kv;
        VrM[k] = vv;
        write_split(r, e, kv);
    }
    if (tid < NS) wc[tid] = tid < n_fill ? 1.f : 0.f;
    if (targets)
        for (int i = tid; i < n_fill; i += blockDim.x) targets[i] = -2;

    // evicted tokens i0 .. i0+nb-1 of a block into token buffer `buf`
    auto fetch_block = [&](int i0, int buf) {
        const int nb = min(NB, n_ev - i0);
        for (int c = tid; c < nb * 2 * CPR; c += blockDim.x) {
            const int tok = c / (2 * CPR), rem = c % (2 * CPR);
            const int which = rem / CPR, cc = rem % CPR;
            const int t = evl[i0 + tok];
            uint8_t *dst = (which ? tokV : tokK) + ((size_t)buf * NB + tok) * ROWB + cc * 16;
            cp_async16(dst, (which ? Vg : Kg) + (size_t)t * ROWB + cc * 16);
        }
        cp_async_commit();
    };

    if (n_fill < n_ev) fetch_block(n_fill, 0);
    int buf = 0;
    for (int i0 = n_fill; i0 < n_ev; i0 += NB, buf ^= 1) {
        const int nb = min(NB, n_ev - i0);
        cp_async_wait<0>();
        __syncthreads();  // this block's tokens have landed; the previous block's update is done
        // next block into the other buffer, whose last readers (the previous block's update) are
        // behind the barrier above; it lands while this block is processed
        if (i0 + NB < n_ev) fetch_block(i0 + NB, buf ^ 1);
        const uint8_t *bK = tokK + (size_t)buf * NB * ROWB;
        const uint8_t *bV = tokV + (size_t)buf * NB * ROWB;

        // ---- bulk: D0 (16 tiles of 16 tokens x 8 slots) and Gm (32 tiles of 16 x 8 tokens) ----
        for (int item = warp; item < 4 * NTD + 32; item += n_warps) {
            const bool is_g = item >= 4 * NTD;
            const int it = is_g ? item - 4 * NTD : item;
            const int mt = is_g ? it / 8 : it / NTD, nt = is_g ? it % 8 : it % NTD;
            if (!is_g && nt * 8 >= Br) continue;
            const uint8_t *pa = bK + (mt * 16 + gq) * ROWB + tig * 16;
            float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
            const int n_split = is_g ? 1 : 3;
            for (int sp = 0; sp < n_split; ++sp) {
                const uint8_t *pb = (is_g ? bK : KrS + (size_t)sp * NS * ROWB) + (nt * 8 + gq) * ROWB + tig * 16;
#pragma unroll
                for (int j = 0; j < SEG; ++j) {
                    const uint4 ra = *reinterpret_cast<const uint4 *>(pa + j * 64);
                    const uint4 rc = *reinterpret_cast<const uint4 *>(pa + 8 * ROWB + j * 64);
                    const uint4 qb = *reinterpret_cast<const uint4 *>(pb + j * 64);
                    mma_16x8x16<T>(c0, ra.x, rc.x, ra.y, rc.y, qb.x, qb.y);
                    mma_16x8x16<T>(c1, ra.z, rc.z, ra.w, rc.w, qb.z, qb.w);
                }
            }
            const int row = mt * 16 + gq, col = nt * 8 + tig * 2;
            if (is_g) {
                Gm[row * kBlkGS + col] = c0[0] + c1[0];
                Gm[row * kBlkGS + col + 1] = c0[1] + c1[1];
                Gm[(row + 8) * kBlkGS + col] = c0[2] + c1[2];
                Gm[(row + 8) * kBlkGS + col + 1] = c0[3] + c1[3];
            } else {
                const float w0a = wc[col], w0b = wc[col + 1];
                Num[row * NS1 + col] = w0a * (c0[0] + c1[0]);
                Num[row * NS1 + col + 1] = w0b * (c0[1] + c1[1]);
                Num[(row + 8) * NS1 + col] = w0a * (c0[2] + c1[2]);
                Num[(row + 8) * NS1 + col + 1] = w0b * (c0[3] + c1[3]);
            }
        }
        __syncthreads();

        // ---- the chain itself, one warp: lane r watches slot r ----
        // The numerators of the current token and the next three live in registers and take
        // their corrections there; shared memory is corrected only from four tokens ahead, so
        // no shared-memory round trip sits between one token's argmax and the next.
        if (warp == 0) {
            // lane l watches slots l, l + 32, ..
            float w[SPL], rw[SPL], rwn[SPL], n0[SPL], n1[SPL], n2[SPL];
#pragma unroll
            for (int s = 0; s < SPL; ++s) {
                const int slot = lane + 32 * s;
                w[s] = slot < Br ? wc[slot] : 1.f;
                rw[s] = __frcp_rn(w[s]);
                rwn[s] = __frcp_rn(w[s] + 1.f);
                n0[s] = Num[slot];
                n1[s] = 1 < nb ? Num[1 * NS1 + slot] : 0.f;
                n2[s] = 2 < nb ? Num[2 * NS1 + slot] : 0.f;
            }
#pragma unroll 4
            for (int t = 0; t < nb; ++t) {
                // independent of this token's outcome: its Gram entries with the next three
                // tokens, and the numerators of the token three ahead
                const float g1 = t + 1 < nb ? Gm[t * kBlkGS + t + 1] : 0.f;
                const float g2 = t + 2 < nb ? Gm[t * kBlkGS + t + 2] : 0.f;
                const float g3 = t + 3 < nb ? Gm[t * kBlkGS + t + 3] : 0.f;
                float n3[SPL];
                uint32_t key[SPL], kmax = 0u;
#pragma unroll
                for (int s = 0; s < SPL; ++s) {
                    const int slot = lane + 32 * s;
                    n3[s] = t + 3 < nb ? Num[(t + 3) * NS1 + slot] : 0.f;
                    key[s] = slot < Br ? order_key(n0[s] * rw[s]) : 0u;  // k_r . k_t  (Eq. (hatr))
                    kmax = key[s] > kmax ? key[s] : kmax;
                }
                const uint32_t best = __reduce_max_sync(0xffffffffu, kmax);
                int rhat = -1;  // equal values go to the lowest slot: slots l before slots l + 32
#pragma unroll
                for (int s = 0; s < SPL; ++s) {
                    const unsigned bal = __ballot_sync(0xffffffffu, key[s] == best && lane + 32 * s < Br);
                    if (rhat < 0 && bal) rhat = 32 * s + __ffs(bal) - 1;
                }
                if (lane == 0) tgt[t] = rhat;
#pragma unroll
                for (int s = 0; s < SPL; ++s) {
                    const bool me = lane + 32 * s == rhat;
                    w[s] += me ? 1.f : 0.f;
                    rw[s] = me ? rwn[s] : rw[s];
                    rwn[s] = __frcp_rn(w[s] + 1.f);
                    n1[s] += me ? g1 : 0.f;
                    n2[s] += me ? g2 : 0.f;
                    n3[s] += me ? g3 : 0.f;
                }
                for (int u = t + 4 + lane; u < nb; u += 32)
                    Num[u * NS1 + rhat] += Gm[t * kBlkGS + u];  // Gm is symmetric: row t
                __syncwarp();
#pragma unroll
                for (int s = 0; s < SPL; ++s) {
                    n0[s] = n1[s];
                    n1[s] = n2[s];
                    n2[s] = n3[s];
                }
            }
        }
        __syncthreads();

        // ---- Eq. (kvr) for the whole block: slot r's mean over its old content and its takes ----
        for (int r = warp; r < Br; r += n_warps) {
            float sk[EPT], sv[EPT];
#pragma unroll
            for (int e = 0; e < EPT; ++e) sk[e] = sv[e] = 0.f;
            int n = 0;
            // which of the block's tokens went to slot r: one vote per half of the block
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int tt = half * 32 + lane;
                unsigned mask = __ballot_sync(0xffffffffu, tt < nb && tgt[tt] == r);
                while (mask) {
                    const int t = half * 32 + __ffs(mask) - 1;
                    mask &= mask - 1;
                    const T *kt = reinterpret_cast<const T *>(bK + (size_t)t * ROWB) + lane * EPT;
                    const T *vt = reinterpret_cast<const T *>(bV + (size_t)t * ROWB) + lane * EPT;
#pragma unroll
                    for (int e = 0; e < EPT; ++e) {
                        sk[e] += E::to_float(kt[e]);
                        sv[e] += E::to_float(vt[e]);
                    }
                    ++n;
                }
            }
            if (n > 0) {
                const float w0 = wc[r];
                const float inv = __frcp_rn(w0 + static_cast<float>(n));
#pragma unroll
                for (int e = 0; e < EPT; ++e) {
                    const int k = r * D + lane * EPT + e;
                    const float nk = fmaf(w0, KrM[k], sk[e]) * inv;
                    KrM[k] = nk;
                    VrM[k] = fmaf(w0, VrM[k], sv[e]) * inv;
                    write_split(r, lane * EPT + e, nk);
                }
                __syncwarp();
                if (lane == 0) wc[r] = w0 + static_cast<float>(n);
            }
        }
        if (targets)
            for (int t = tid; t < nb; t += blockDim.x) targets[i0 + t] = tgt[t];
        // the next iteration's barrier orders these writes before their readers
    }
    __syncthreads();

    const int n_res = n_fill;
    float *Kr_g = reinterpret_cast<float *>(p.base + d.kr_off);
    float *Vr_g = reinterpret_cast<float *>(p.base + d.vr_off);
    uint32_t *w_g = reinterpret_cast<uint32_t *>(p.base + d.w_off);
    for (int k = tid; k < n_res * D; k += blockDim.x) {
        Kr_g[k] = KrM[k];
        Vr_g[k] = VrM[k];
    }
    for (int k = tid; k < n_res; k += blockDim.x) w_g[k] = static_cast<uint32_t>(wc[k]);
}

// ---------------------------------------------------------------------------
// P5: survivors into the unit's slots, ascending position; one warp per row.
// ---------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(256) prefill_gather_kernel(const PrefillParams p, const float *scores) {
    constexpr int ROWB = D * (int)sizeof(T);
    constexpr int CPR = ROWB / 16;
    const int ul = blockIdx.y;
    const UnitDesc d = p.desc[ul];
    const int T_len = p.T;
    const int32_t *cnt = reinterpret_cast<const int32_t *>(p.ws + p.wl.counts) + ul * 4;
    const int n_ev = cnt[0], n_kept = cnt[1];
    const int cap = d.Bp + d.Bc;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (n_kept > cap) dev_set_status(p.status, DEV_ERR_CHECK, d.unit, 4);
        UnitCounters c;
        c.n_live = min(n_kept, cap);
        c.n_res = min(d.Br, n_ev);
        c.T = T_len;
        c.pad = 0;
        p.counters[d.unit] = c;
    }
    const int row = blockIdx.x * 8 + warp;
    if (row >= min(n_kept, cap)) return;
    const int t = reinterpret_cast<const int32_t *>(p.ws + p.wl.kept_list)[(size_t)ul * T_len + row];
    const uint4 *ks = reinterpret_cast<const uint4 *>(static_cast<const uint8_t *>(p.K) + ((size_t)ul * T_len + t) * ROWB);
    const uint4 *vs = reinterpret_cast<const uint4 *>(static_cast<const uint8_t *>(p.V) + ((size_t)ul * T_len + t) * ROWB);
    uint4 *kd = reinterpret_cast<uint4 *>(p.base + d.k_off + (size_t)row * ROWB);
    uint4 *vd = reinterpret_cast<uint4 *>(p.base + d.v_off + (size_t)row * ROWB);
    for (int c = lane; c < CPR; c += 32) {
        kd[c] = ks[c];
        vd[c] = vs[c];
    }
    if (lane == 0) {
        reinterpret_cast<float *>(p.base + d.score_off)[row] = scores[(size_t)ul * T_len + t];
        reinterpret_cast<int32_t *>(p.base + d.pos_off)[row] = t;
    }
}

template <int D>
size_t merge_smem_bytes(int Br, int row_bytes) {
    const int br_pad = (Br + 3) & ~3;
    return (size_t)Br * D * 8 + (size_t)br_pad * 8 + (size_t)(kMergeIB + kMergePF) * 4 +
           (size_t)kMergePF * 2 * row_bytes;
}

template <typename T, int D>
int launch_all(const PrefillParams &p, int max_br, cudaStream_t stream) {
    const int n_chunks = (p.T + kPrefillChunk - 1) / kPrefillChunk;
    const float *scores = p.scores_in;
    if (p.Qw) {
        const size_t sm = (size_t)(kPrefillChunk + kQB) * (D + 4) * 4;
        if constexpr (sizeof(T) == 2)
        {
            // at most two CTAs per SM over the whole launch -- one wave -- each walking its share
            // of a unit's chunks
            const int per_unit = std::max(1, std::min(n_chunks, (2 * p.n_sm) / p.units));
            const int GW = p.G * p.W;
            if (window_logits_tc_supported(GW)) {
                // windows of 32 .. 128 query rows: the tcgen05 form
                WindowLogitsParams wp;
                wp.K = p.K;
                wp.Qw = p.Qw;
                wp.logits = reinterpret_cast<float *>(p.ws + p.wl.logits);
                wp.partial = reinterpret_cast<float2 *>(p.ws + p.wl.partial);
                wp.status = p.status;
                wp.units = p.units;
                wp.n_kv_heads = p.n_kv_heads;
                wp.T = p.T;
                wp.W = p.W;
                wp.G = p.G;
                wp.scale = p.scale;
                // two CTAs fit an SM up to 64 rows, one beyond (the window's rows are resident)
                const int ctas = GW <= 64 ? 2 * p.n_sm : p.n_sm;
                const int px = std::max(1, std::min(n_chunks, ctas / p.units));
                const int rc = launch_window_logits_tc(Elem<T>::kIsBf16 ? 2 : 1, D, wp, px, stream);
                if (rc != 0) return rc;
            } else
                prefill_logits_mma_kernel<T, D><<<dim3(per_unit, p.units), kP1Threads, logits_mma_smem_bytes<D>(), stream>>>(p);
        }
        else
            prefill_logits_kernel<T, D><<<dim3(n_chunks, p.units), 256, sm, stream>>>(p);
        const int rows = p.units * p.G * p.W;
        prefill_rowstat_kernel<<<(rows + 127) / 128, 128, 0, stream>>>(p, n_chunks);
        prefill_scores_kernel<<<dim3((p.T + 255) / 256, p.units), 256, 0, stream>>>(p);
        scores = reinterpret_cast<const float *>(p.ws + p.wl.scores);
    }
    prefill_select_kernel<<<p.units, 1024, 0, stream>>>(p, scores);
    // the residual chain: merged rows in registers, one per warp, up to 128 merged slots (one
    // warp per unit when the layer has many units); the shared-memory form beyond
    if (p.cosine)  // the cosine variant of Eq. (hatr) is built into the general form only
        prefill_merge_kernel<T, D><<<p.units, kMergeWarps * 32,
                                     merge_smem_bytes<D>(max_br, D * (int)sizeof(T)), stream>>>(p);
    else if (max_br <= 32 && p.units > 2 * p.n_sm)  // more chains than the CTA forms fit at once
        prefill_merge_warp_kernel<T, D><<<p.units, 32, merge_warp_smem_bytes<T, D>(), stream>>>(p);
    else if (max_br <= 32 && sizeof(T) == 2) {
        if constexpr (sizeof(T) == 2)
            prefill_merge_blocked_kernel<T, D, 32><<<p.units, 1024, BlkSmem<D, 32>::total, stream>>>(p);
    } else if (max_br <= 64 && sizeof(T) == 2 && p.units <= 2 * p.n_sm) {
        if constexpr (sizeof(T) == 2)
            prefill_merge_blocked_kernel<T, D, 64><<<p.units, 1024, BlkSmem<D, 64>::total, stream>>>(p);
    } else if (max_br <= 32)
        prefill_merge_rows_kernel<T, D, 1><<<p.units, kRowMergeThreads, merge_rows_smem_bytes<T, D>(), stream>>>(p);
    else if (max_br <= 64)
        prefill_merge_rows_kernel<T, D, 2><<<p.units, kRowMergeThreads, merge_rows_smem_bytes<T, D>(), stream>>>(p);
    else if (max_br <= 128)
        prefill_merge_rows_kernel<T, D, 4><<<p.units, kRowMergeThreads, merge_rows_smem_bytes<T, D>(), stream>>>(p);
    else
        prefill_merge_kernel<T, D><<<p.units, kMergeWarps * 32,
                                     merge_smem_bytes<D>(max_br, D * (int)sizeof(T)), stream>>>(p);
    // the largest unit bounds the gather grid; rows past a unit's survivors return at once
    const int max_rows = p.max_cap < p.T ? p.max_cap : p.T;
    prefill_gather_kernel<T, D><<<dim3((max_rows + 7) / 8, p.units), 256, 0, stream>>>(p, scores);
    return static_cast<int>(cudaGetLastError());
}

template <typename T, int D>
int prepare_all() {
    if constexpr (sizeof(T) == 2) {
        cudaError_t e2 = cudaFuncSetAttribute(prefill_logits_mma_kernel<T, D>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)logits_mma_smem_bytes<D>());
        if (e2 != cudaSuccess) return static_cast<int>(e2);
    }
    cudaError_t e = cudaFuncSetAttribute(prefill_logits_kernel<T, D>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)((kPrefillChunk + kQB) * (D + 4) * 4));
    if (e != cudaSuccess) return static_cast<int>(e);
    e = cudaFuncSetAttribute(prefill_merge_kernel<T, D>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)merge_smem_bytes<D>(prefill_max_residual(D), D * (int)sizeof(T)));
    if (e != cudaSuccess) return static_cast<int>(e);
    if constexpr (sizeof(T) == 2) {
        e = cudaFuncSetAttribute(prefill_merge_blocked_kernel<T, D, 32>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BlkSmem<D, 32>::total);
        if (e != cudaSuccess) return static_cast<int>(e);
        e = cudaFuncSetAttribute(prefill_merge_blocked_kernel<T, D, 64>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BlkSmem<D, 64>::total);
        if (e != cudaSuccess) return static_cast<int>(e);
    }
    e = cudaFuncSetAttribute(prefill_merge_warp_kernel<T, D>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)merge_warp_smem_bytes<T, D>());
    return static_cast<int>(e);
}

}  // namespace

int prefill_max_residual(int D) { return (192 * 1024) / (D * 8); }

int launch_prefill(int dtype, int D, const PrefillParams &p, int max_br, cudaStream_t stream) {
    if (dtype == 0 && D == 64) return launch_all<float, 64>(p, max_br, stream);
    if (dtype == 0 && D == 128) return launch_all<float, 128>(p, max_br, stream);
    if (dtype == 1 && D == 64) return launch_all<__half, 64>(p, max_br, stream);
    if (dtype == 1 && D == 128) return launch_all<__half, 128>(p, max_br, stream);
    if (dtype == 2 && D == 64) return launch_all<__nv_bfloat16, 64>(p, max_br, stream);
    if (dtype == 2 && D == 128) return launch_all<__nv_bfloat16, 128>(p, max_br, stream);
    return -1;
}

int prepare_prefill(int dtype, int D) {
    if (dtype == 0 && D == 64) return prepare_all<float, 64>();
    if (dtype == 0 && D == 128) return prepare_all<float, 128>();
    if (dtype == 1 && D == 64) return prepare_all<__half, 64>();
    if (dtype == 1 && D == 128) return prepare_all<__half, 128>();
    if (dtype == 2 && D == 64) return prepare_all<__nv_bfloat16, 64>();
    if (dtype == 2 && D == 128) return prepare_all<__nv_bfloat16, 128>();
    return -1;
}

}  // namespace zsm
