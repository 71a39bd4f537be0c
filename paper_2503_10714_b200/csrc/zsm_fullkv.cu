// Decode attention over an UNCOMPRESSED cache (Eq. (att_score), Sec. 3.1): the same-hardware
// counterpart of the paper's FullKV baseline, for the cache path only.
//
// A head's T tokens are cut into chunks; one work item = (unit, chunk).  Persistent CTAs take
// items round-robin and stream each through the same shared-memory ring as the compressed
// path (producer warp: 1-D bulk copies + mbarriers; eight consumer warps): K tiles -> logits on
// the tensor cores (mma.sync m16n8k16) -> chunk maximum and exponentials -> V tiles -> the
// chunk's partial (max, sum, unnormalised output).  A second small kernel folds a head's
// partials into the output.  16-bit storage only.
#include "../../include/zsm.h"

#include "zsm_common.cuh"

namespace zsm {

namespace {

constexpr int kFkTile = 16384;   // ring stage
constexpr int kFkWarps = 8;      // consumer warps (+ 1 producer warp)
constexpr int kFkThreads = (kFkWarps + 1) * 32;
constexpr int kFkSmemPerCta = 232448 / 2 - 1024;  // two CTAs per SM
constexpr int kFkWsHeader = 256;  // status word at the head of the workspace

struct FullKvParams {
    const uint8_t *K, *V, *q;  // [units][T][d], [units][T][d], [units][G][d]
    float *part;               // [items][G][d + 2]: max, sum, unnormalised output
    int32_t *status;
    int32_t n_units, T, chunk, n_chunks, stages;
    float scale;
};

struct FkSmem {
    uint32_t ring, bars, flags, probs, opart, redf, total;
};

__host__ __device__ inline FkSmem fk_smem_layout(int stages, int G, int D, int chunk) {
    FkSmem L;
    uint32_t o = 0;
    auto take = [&](uint32_t bytes) {
        uint32_t at = o;
        o += (bytes + 127u) & ~127u;
        return at;
    };
    L.ring = take(static_cast<uint32_t>(stages) * kFkTile);
    L.bars = take(2u * static_cast<uint32_t>(stages) * 8u);
    L.flags = take(64u);
    L.probs = take(static_cast<uint32_t>(chunk) * G * 4u);
    L.opart = take(static_cast<uint32_t>(kFkWarps) * G * D * 4u);
    L.redf = take(2u * kFkWarps * 8u * 4u);
    L.total = o;
    return L;
}

enum : int32_t { FW_PRODUCER = 21, FW_HEADER = 22, FW_K = 23, FW_V = 24 };

template <typename T, int D, int G>
__global__ void __launch_bounds__(kFkThreads, 2) fullkv_chunk_kernel(const FullKvParams p) {
    using E = Elem<T>;
    constexpr int EPL = E::EPL;
    constexpr int EP2 = EPL / 2;
    constexpr int ROWB = D * (int)sizeof(T);
    constexpr int LPR = D / EPL;
    constexpr int RPW = 32 / LPR;
    constexpr int R = kFkTile / ROWB;
    constexpr int SEG = ROWB / 64;
    constexpr int RB = R / 16;
    constexpr int UBV = G <= 4 ? 4 : 2;
    constexpr int NW = kFkWarps, NT = NW * 32;
    static_assert(sizeof(T) == 2, "16-bit storage only");

    extern __shared__ __align__(128) uint8_t smem[];
    const int S = p.stages;
    const FkSmem L = fk_smem_layout(S, G, D, p.chunk);
    uint8_t *ring = smem + L.ring;
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + L.bars);
    uint64_t *empty_bar = full_bar + S;
    volatile int32_t *abort_flag = reinterpret_cast<volatile int32_t *>(smem + L.flags);
    float *probs = reinterpret_cast<float *>(smem + L.probs);  // [row][G]
    float *opart = reinterpret_cast<float *>(smem + L.opart);
    float *redf = reinterpret_cast<float *>(smem + L.redf);
    float *redf2 = redf + NW * 8;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], NW);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const int n_items = p.n_units * p.n_chunks;

    // ---------------- producer ----------------
    if (warp == NW) {
        if (lane != 0) return;
        int s = 0;
        uint32_t ph = 0;
        auto acquire = [&](uint32_t bytes, uint64_t *&bar) -> uint8_t * {
            if (!mbar_wait_bounded(&empty_bar[s], ph ^ 1u, abort_flag, p.status, FW_PRODUCER))
                return nullptr;
            bar = &full_bar[s];
            mbar_arrive_expect_tx(bar, bytes);
            uint8_t *dst = ring + static_cast<size_t>(s) * kFkTile;
            if (++s == S) {
                s = 0;
                ph ^= 1u;
            }
            return dst;
        };
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const int u = item / p.n_chunks, c = item % p.n_chunks;
            const int row_lo = c * p.chunk, rows = min(p.chunk, p.T - row_lo);
            uint64_t *bar = nullptr;
            uint8_t *dst = acquire(G * ROWB, bar);
            if (!dst) break;
            bulk_g2s(dst, p.q + (size_t)u * G * ROWB, G * ROWB, bar);
            for (int pass = 0; pass < 2 && ok; ++pass) {
                const uint8_t *src = (pass ? p.V : p.K) + ((size_t)u * p.T + row_lo) * ROWB;
                for (int r0 = 0; r0 < rows; r0 += R) {
                    const uint32_t bytes = static_cast<uint32_t>(min(R, rows - r0)) * ROWB;
                    dst = acquire(bytes, bar);
                    if (!dst) {
                        ok = false;
                        break;
                    }
                    bulk_g2s(dst, src + (size_t)r0 * ROWB, bytes, bar);
                }
            }
        }
        if (!ok) {
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
        return;
    }

    // ---------------- consumers ----------------
    const int l = lane % LPR, sub = lane / LPR;
    const int gq = lane >> 2, tig = lane & 3;
    int cs = 0;
    uint32_t cph = 0;
    auto wait_full = [&](int where) -> const uint8_t * {
        if (!mbar_wait_bounded(&full_bar[cs], cph, abort_flag, p.status, where)) return nullptr;
        return ring + static_cast<size_t>(cs) * kFkTile;
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
    constexpr int rb_step = RB % NW;

    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int c = item % p.n_chunks;
        const int n_rows = min(p.chunk, p.T - c * p.chunk);

        // header: the group's queries as B fragments (head n = lane / 4; heads >= G are zero)
        const uint8_t *h = wait_full(FW_HEADER);
        if (!h) return;
        uint32_t qb[SEG][4];
#pragma unroll
        for (int j = 0; j < SEG; ++j) {
            uint4 t = make_uint4(0, 0, 0, 0);
            if (gq < G) t = *reinterpret_cast<const uint4 *>(h + gq * ROWB + j * 64 + tig * 16);
            qb[j][0] = t.x;
            qb[j][1] = t.y;
            qb[j][2] = t.z;
            qb[j][3] = t.w;
        }
        release();

        // logits: blocks of 16 rows go round the warps; maxima of this thread's two heads
        float tmax0 = -INFINITY, tmax1 = -INFINITY;
        int kturn = 0;
        for (int r0 = 0; r0 < n_rows; r0 += R) {
            const uint8_t *tile = wait_full(FW_K);
            if (!tile) return;
            const int rows = min(R, n_rows - r0);
            int rb_first = warp - kturn;
            if (rb_first < 0) rb_first += NW;
            for (int rb = rb_first; rb < RB && rb * 16 < rows; rb += NW) {
                const uint8_t *pa = tile + (rb * 16 + gq) * ROWB + tig * 16;
                float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int j = 0; j < SEG; ++j) {
                    const uint4 ra = *reinterpret_cast<const uint4 *>(pa + j * 64);
                    const uint4 rc = *reinterpret_cast<const uint4 *>(pa + 8 * ROWB + j * 64);
                    mma_16x8x16<T>(c0, ra.x, rc.x, ra.y, rc.y, qb[j][0], qb[j][1]);
                    mma_16x8x16<T>(c1, ra.z, rc.z, ra.w, rc.w, qb[j][2], qb[j][3]);
                }
                const int n0 = tig * 2;
                if (n0 < G) {
                    const int ra_ = rb * 16 + gq, rc_ = ra_ + 8;
                    float *pr = probs + (r0 + ra_) * G + n0;
                    if (ra_ < rows) {
                        const float x0 = (c0[0] + c1[0]) * p.scale;
                        pr[0] = x0;
                        tmax0 = fmaxf(tmax0, x0);
                        if (G > 1) {
                            const float x1 = (c0[1] + c1[1]) * p.scale;
                            pr[1] = x1;
                            tmax1 = fmaxf(tmax1, x1);
                        }
                    }
                    if (rc_ < rows) {
                        const float x0 = (c0[2] + c1[2]) * p.scale;
                        pr[8 * G] = x0;
                        tmax0 = fmaxf(tmax0, x0);
                        if (G > 1) {
                            const float x1 = (c0[3] + c1[3]) * p.scale;
                            pr[8 * G + 1] = x1;
                            tmax1 = fmaxf(tmax1, x1);
                        }
                    }
                }
            }
            kturn += rb_step;
            if (kturn >= NW) kturn -= NW;
            release();
        }

        // chunk maximum per head, then exponentials and their sum
        float mx[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            mx[g] = -INFINITY;
            if (g == tig * 2) mx[g] = tmax0;
            if (g == tig * 2 + 1) mx[g] = tmax1;
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
            for (int j = tid; j < n_rows; j += NT) {
                float pv[G];
                load_group<G>(probs + j * G, pv);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    pv[g] = expf(pv[g] - mx[g]);
                    sm[g] += pv[g];
                }
                store_group<G>(probs + j * G, pv);
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                sm[g] = group_sum<32>(sm[g]);
                if (lane == 0) redf2[warp * G + g] = sm[g];
            }
        }
        csync();

        // output pass
        float2 acc2[G][EP2];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int e = 0; e < EP2; ++e) acc2[g][e] = make_float2(0.f, 0.f);
        for (int r0 = 0; r0 < n_rows; r0 += R) {
            const uint8_t *tile = wait_full(FW_V);
            if (!tile) return;
            const int rows = min(R, n_rows - r0);
            for (int base = warp * RPW; base < rows; base += NW * RPW * UBV) {
                uint4 raw[UBV];
#pragma unroll
                for (int u = 0; u < UBV; ++u) {
                    const int row = base + u * NW * RPW + sub;
                    raw[u] = row < rows ? *reinterpret_cast<const uint4 *>(tile + row * ROWB + l * 16)
                                        : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int u = 0; u < UBV; ++u) {
                    const int row = base + u * NW * RPW + sub;
                    float f[EPL];
                    E::widen(raw[u], f);
                    float pv[G];
                    if (row < rows) {
                        load_group<G>(probs + (r0 + row) * G, pv);
                    } else {
#pragma unroll
                        for (int g = 0; g < G; ++g) pv[g] = 0.f;
                    }
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const float2 pp = make_float2(pv[g], pv[g]);
#pragma unroll
                        for (int e = 0; e < EP2; ++e)
                            acc2[g][e] = __ffma2_rn(pp, make_float2(f[2 * e], f[2 * e + 1]), acc2[g][e]);
                    }
                }
            }
            release();
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                float v = (e & 1) ? acc2[g][e / 2].y : acc2[g][e / 2].x;
#pragma unroll
                for (int off = LPR; off < 32; off <<= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
                if (sub == 0) opart[(warp * G + g) * D + l * EPL + e] = v;
            }
        }
        csync();
        float *part = p.part + (size_t)item * G * (D + 2);
        for (int k = tid; k < G * D; k += NT) {
            const int g = k / D, dim = k % D;
            float sum = 0.f;
            for (int wv = 0; wv < NW; ++wv) sum += opart[(wv * G + g) * D + dim];
            part[g * (D + 2) + 2 + dim] = sum;
        }
        if (tid < G) {
            float m = redf[tid], z = 0.f;
            for (int wv = 1; wv < NW; ++wv) m = fmaxf(m, redf[wv * G + tid]);
            for (int wv = 0; wv < NW; ++wv) z += redf2[wv * G + tid];
            part[tid * (D + 2)] = m;
            part[tid * (D + 2) + 1] = z;
        }
        csync();  // shared scratch is free for the next item
    }
}

// Folds a head's chunk partials: one block per (unit, query head), one thread per dimension.
template <typename T>
__global__ void fullkv_combine_kernel(const float *part, T *out, int n_chunks, int G, int D) {
    const int ug = blockIdx.x;  // unit * G + g
    const int u = ug / G, g = ug % G, dim = threadIdx.x;
    if (dim >= D) return;
    const size_t stride = (size_t)G * (D + 2);
    const float *p0 = part + (size_t)u * n_chunks * stride + (size_t)g * (D + 2);
    float M = -INFINITY;
    for (int c = 0; c < n_chunks; ++c) M = fmaxf(M, p0[c * stride]);
    float Z = 0.f, o = 0.f;
    for (int c = 0; c < n_chunks; ++c) {
        const float w = expf(p0[c * stride] - M);
        Z = fmaf(p0[c * stride + 1], w, Z);
        o = fmaf(p0[c * stride + 2 + dim], w, o);
    }
    out[(size_t)ug * D + dim] = Elem<T>::from_float(o / Z);
}

int chunk_rows(int G) { return 4096 / G; }  // 16 KiB of weights per CTA

template <typename T, int D, int G>
int launch_fullkv(FullKvParams p, void *out, int n_sm, cudaStream_t stream) {
    p.chunk = chunk_rows(G);
    p.n_chunks = (p.T + p.chunk - 1) / p.chunk;
    int stages = 12;
    while (stages > 2 && (int)fk_smem_layout(stages, G, D, p.chunk).total > kFkSmemPerCta) --stages;
    const FkSmem L = fk_smem_layout(stages, G, D, p.chunk);
    if ((int)L.total > kFkSmemPerCta) return -1;
    p.stages = stages;
    cudaError_t e = cudaFuncSetAttribute(fullkv_chunk_kernel<T, D, G>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kFkSmemPerCta);
    if (e != cudaSuccess) return static_cast<int>(e);
    const int n_items = p.n_units * p.n_chunks;
    const int grid = n_items < 2 * n_sm ? n_items : 2 * n_sm;
    fullkv_chunk_kernel<T, D, G><<<grid, kFkThreads, L.total, stream>>>(p);
    fullkv_combine_kernel<T><<<p.n_units * G, D, 0, stream>>>(p.part, static_cast<T *>(out), p.n_chunks, G, D);
    return static_cast<int>(cudaGetLastError());
}

template <typename T>
int dispatch_fullkv(int D, int G, const FullKvParams &p, void *out, int n_sm, cudaStream_t stream) {
#define ZSM_FK(DD, GG) \
    if (D == DD && G == GG) return launch_fullkv<T, DD, GG>(p, out, n_sm, stream);
    ZSM_FK(64, 1) ZSM_FK(64, 2) ZSM_FK(64, 4) ZSM_FK(64, 8)
    ZSM_FK(128, 1) ZSM_FK(128, 2) ZSM_FK(128, 4) ZSM_FK(128, 8)
#undef ZSM_FK
    return -1;
}

bool fk_shape_ok(int32_t n_units, int32_t group, int32_t head_dim, int32_t T) {
    return n_units >= 1 && T >= 1 && (group == 1 || group == 2 || group == 4 || group == 8) &&
           (head_dim == 64 || head_dim == 128);
}

}  // namespace

}  // namespace zsm

using namespace zsm;

extern "C" {

zsm_status_t zsm_fullkv_workspace_bytes(int32_t n_units, int32_t group, int32_t head_dim, int32_t T,
                                        size_t *bytes) {
    if (!bytes || n_units < 1 || T < 1 || group < 1 || head_dim < 1) return ZSM_ERR_INVALID_ARG;
    if (!fk_shape_ok(n_units, group, head_dim, T)) return ZSM_ERR_UNSUPPORTED;
    const size_t n_chunks = ((size_t)T + chunk_rows(group) - 1) / chunk_rows(group);
    *bytes = kFkWsHeader + (size_t)n_units * n_chunks * group * (head_dim + 2) * 4;
    return ZSM_OK;
}

zsm_status_t zsm_fullkv_decode(int32_t dtype, int32_t n_units, int32_t group, int32_t head_dim,
                               int32_t T, const void *K, const void *V, const void *q, void *out,
                               float softmax_scale, void *workspace, size_t workspace_bytes,
                               zsm_stream_t stream) {
    if (!K || !V || !q || !out || !workspace || n_units < 1 || T < 1 || group < 1 || head_dim < 1 ||
        !(softmax_scale >= 0.f))
        return ZSM_ERR_INVALID_ARG;
    if (dtype != ZSM_F16 && dtype != ZSM_BF16) return dtype == ZSM_F32 ? ZSM_ERR_UNSUPPORTED : ZSM_ERR_INVALID_ARG;
    size_t need = 0;
    const zsm_status_t st = zsm_fullkv_workspace_bytes(n_units, group, head_dim, T, &need);
    if (st != ZSM_OK) return st;
    if (workspace_bytes < need) return ZSM_ERR_BUFFER_TOO_SMALL;
    const uintptr_t al = reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V) |
                         reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out);
    if ((al & 15u) != 0 || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return ZSM_ERR_INVALID_ARG;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return ZSM_ERR_CUDA;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace, 0, kFkWsHeader, cs) != cudaSuccess) return ZSM_ERR_CUDA;
    FullKvParams p;
    p.K = static_cast<const uint8_t *>(K);
    p.V = static_cast<const uint8_t *>(V);
    p.q = static_cast<const uint8_t *>(q);
    p.status = static_cast<int32_t *>(workspace);
    p.part = reinterpret_cast<float *>(static_cast<uint8_t *>(workspace) + kFkWsHeader);
    p.n_units = n_units;
    p.T = T;
    p.chunk = p.n_chunks = p.stages = 0;
    p.scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
    const int rc = dtype == ZSM_F16 ? dispatch_fullkv<__half>(head_dim, group, p, out, n_sm, cs)
                                    : dispatch_fullkv<__nv_bfloat16>(head_dim, group, p, out, n_sm, cs);
    if (rc == -1) return ZSM_ERR_UNSUPPORTED;
    return rc == 0 ? ZSM_OK : ZSM_ERR_CUDA;
}

zsm_status_t zsm_fullkv_status(void *workspace, zsm_stream_t stream) {
    if (!workspace) return ZSM_ERR_INVALID_ARG;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return ZSM_ERR_CUDA;
    int32_t st = 0;
    if (cudaMemcpy(&st, workspace, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return ZSM_ERR_CUDA;
    if (st == DEV_ERR_TIMEOUT) return ZSM_ERR_TIMEOUT;
    return st == 0 ? ZSM_OK : ZSM_ERR_DEVICE_CHECK;
}

}  // extern "C"
