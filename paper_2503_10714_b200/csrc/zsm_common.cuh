// Shared device-side definitions of the compressed-KV decode path (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace zsm {

// ---------------------------------------------------------------------------
// Cache layout in device memory.
//
// One unit = one (layer, sequence, kv-head).  Its arrays, all inside the
// caller's buffer and addressed by byte offsets from the buffer base:
//   K, V     token rows  [n_tok][d]   storage dtype, n_tok = B_p + B_c
//   score    fp32 [n_tok_pad]         contribution score, Eq. (score)
//   pos      int32 [n_tok_pad]        sequence position of the slot's token
//   Kr, Vr   residual rows [B_r][d]   fp32 masters of the merged slots, Eq. (kvr)
//   w        uint32 [B_r_pad]         fusion counts
// The pool has no physical split between proximity and context: a token is in
// proximity iff its position is among the B_p highest.  Live rows are packed at
// the front (rows 0..n_live-1); the new token overwrites the evicted row.
// *_pad: rounded up to 4 entries so that 16-byte bulk copies never leave the array.
// ---------------------------------------------------------------------------
struct __align__(16) UnitDesc {
    uint64_t k_off, v_off;
    uint64_t kr_off, vr_off;
    uint64_t score_off, pos_off;
    uint64_t w_off;
    int32_t unit;  // global unit index: (layer*batch + b)*n_kv_heads + h
    int32_t Bp;
    int32_t Bc;
    int32_t Br;
    int32_t pad0, pad1;
};
static_assert(sizeof(UnitDesc) == 80, "UnitDesc is read as five 16-byte words");

// Per-unit dynamic state, one int4 per unit.
struct __align__(16) UnitCounters {
    int32_t n_live;  // token slots in use
    int32_t n_res;   // residual slots in use
    int32_t T;       // tokens seen = position of the next token
    int32_t pad;
};

// Sticky device status: word 0 = first error code, words 1..3 = detail.
enum : int32_t {
    DEV_OK = 0,
    DEV_ERR_CHECK = 6,    // == ZSM_ERR_DEVICE_CHECK
    DEV_ERR_TIMEOUT = 7,  // == ZSM_ERR_TIMEOUT
};

__device__ __forceinline__ void dev_set_status(int32_t *status, int32_t code, int32_t d0,
                                               int32_t d1) {
    if (atomicCAS(status, DEV_OK, code) == DEV_OK) {
        status[1] = d0;
        status[2] = d1;
    }
}

// Monotone map fp32 -> uint32: a < b as floats  <=>  score_order_bits(a) < score_order_bits(b)
// as unsigned integers, for every sign (-0.0 is taken as +0.0 first, so the two zeros tie as
// they do in a float comparison).  The victim search orders 64-bit keys (these bits, position).
__device__ __forceinline__ uint32_t score_order_bits(float s) {
    const uint32_t u = __float_as_uint(s + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// ---------------------------------------------------------------------------
// Storage-type helpers: 16 bytes = EPL elements, widened to fp32.
// ---------------------------------------------------------------------------
template <typename T>
struct Elem;

template <>
struct Elem<float> {
    static constexpr int EPL = 4;
    static constexpr bool kIsBf16 = false;
    __device__ static __forceinline__ void widen(const uint4 &raw, float (&f)[4]) {
        f[0] = __uint_as_float(raw.x);
        f[1] = __uint_as_float(raw.y);
        f[2] = __uint_as_float(raw.z);
        f[3] = __uint_as_float(raw.w);
    }
    __device__ static __forceinline__ float to_float(float x) { return x; }
    __device__ static __forceinline__ float from_float(float x) { return x; }
};

template <>
struct Elem<__half> {
    static constexpr int EPL = 8;
    static constexpr bool kIsBf16 = false;
    __device__ static __forceinline__ void widen(const uint4 &raw, float (&f)[8]) {
        const __half2 *h = reinterpret_cast<const __half2 *>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 t = __half22float2(h[i]);
            f[2 * i] = t.x;
            f[2 * i + 1] = t.y;
        }
    }
    __device__ static __forceinline__ float to_float(__half x) { return __half2float(x); }
    __device__ static __forceinline__ __half from_float(float x) { return __float2half_rn(x); }
};

template <>
struct Elem<__nv_bfloat16> {
    static constexpr int EPL = 8;
    static constexpr bool kIsBf16 = true;
    __device__ static __forceinline__ void widen(const uint4 &raw, float (&f)[8]) {
        const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(u[i] << 16);
            f[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
        }
    }
    __device__ static __forceinline__ float to_float(__nv_bfloat16 x) {
        return __bfloat162float(x);
    }
    __device__ static __forceinline__ __nv_bfloat16 from_float(float x) {
        return __float2bfloat16_rn(x);
    }
};

// ---------------------------------------------------------------------------
// mbarrier / bulk-copy primitives (own CTA's shared memory, own GPU's memory,
// never a multicast form).
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// The same test, but the thread may stay suspended for up to `hint_ns` (a hint; the hardware
// caps it) or until the phase completes, instead of returning at once: a waiting warp then
// issues a poll now and then rather than spinning.
__device__ __forceinline__ bool mbar_try_wait_suspend(uint64_t *bar, uint32_t parity,
                                                      uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false when the wait was given up: either this thread
// waited longer than the limit (it then records ZSM_ERR_TIMEOUT and raises the
// CTA's abort flag) or another thread of the CTA already gave up.  A barrier
// whose phase has completed always returns true, whatever the abort flag says,
// so every thread of a CTA stops at the same point of the tile sequence.
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s
constexpr uint32_t kSuspendHintNs = 20000u;        // per poll

__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity,
                                                  volatile int32_t *abort_flag, int32_t *status,
                                                  int32_t where, uint64_t limit_ns = kWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    uint32_t polls = 0;
    while (true) {
        if (mbar_try_wait_suspend(bar, parity, kSuspendHintNs)) return true;
        ++polls;
        if ((polls & 7u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > limit_ns) {
                dev_set_status(status, DEV_ERR_TIMEOUT, where, static_cast<int32_t>(blockIdx.x));
                *abort_flag = 1;
                __threadfence_block();
                return false;
            }
        }
    }
}

// 1-D bulk copy global -> this CTA's shared memory, completion on an mbarrier.
// Both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void *smem_dst, const void *gmem_src, uint32_t bytes,
                                         uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_u32(smem_dst)),
        "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// ---------------------------------------------------------------------------
// Small device helpers shared by the attention kernels.
// ---------------------------------------------------------------------------
template <int LANES>
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
    for (int off = LANES / 2; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// G consecutive floats (one slot's weights for the whole group).
template <int G>
__device__ __forceinline__ void load_group(const float *p, float (&v)[G]) {
    if constexpr (G == 1) {
        v[0] = p[0];
    } else if constexpr (G == 2) {
        const float2 t = *reinterpret_cast<const float2 *>(p);
        v[0] = t.x;
        v[1] = t.y;
    } else {
#pragma unroll
        for (int i = 0; i < G / 4; ++i) {
            const float4 t = reinterpret_cast<const float4 *>(p)[i];
            v[4 * i] = t.x;
            v[4 * i + 1] = t.y;
            v[4 * i + 2] = t.z;
            v[4 * i + 3] = t.w;
        }
    }
}

template <int G>
__device__ __forceinline__ void store_group(float *p, const float (&v)[G]) {
    if constexpr (G == 1) {
        p[0] = v[0];
    } else if constexpr (G == 2) {
        *reinterpret_cast<float2 *>(p) = make_float2(v[0], v[1]);
    } else {
#pragma unroll
        for (int i = 0; i < G / 4; ++i)
            reinterpret_cast<float4 *>(p)[i] =
                make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    }
}

// One m16n8k16 tensor-core step with fp32 accumulation: c += A(16 x 16, row-major) * B(16 x 8).
// a0..a3 and b0, b1 are packed pairs of 16-bit elements in the instruction's fragment order.
template <typename T>
__device__ __forceinline__ void mma_16x8x16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                            uint32_t a3, uint32_t b0, uint32_t b1) {
    if constexpr (sizeof(T) == 2 && Elem<T>::kIsBf16) {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
            "{%8,%9}, {%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    } else {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
            "{%8,%9}, {%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    }
}

}  // namespace zsm
