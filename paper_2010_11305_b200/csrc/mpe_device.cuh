// Device-side building blocks: counter hash, set hash, row loads, the row-wise
// min-max quantizer with nearest-even or stochastic rounding (Section 3
// "Precision"/"Rounding", Algorithm 1).  Every FP32 operation that feeds a stored
// code is spelled with an explicit rounding intrinsic so that the compiler can
// neither contract nor reorder it.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mpe {

constexpr uint32_t DOMAIN_INIT = 1, DOMAIN_SR = 2, DOMAIN_FLUSH = 3;
constexpr int LOC_MISS = -1;      // unique row not cache resident
constexpr int LOC_INVALID = -2;   // pseudo row collecting out-of-range indices

__host__ __device__ __forceinline__ uint32_t mix32(uint32_t x) {
    x ^= x >> 16; x *= 0x7feb352dU; x ^= x >> 15; x *= 0x846ca68bU; x ^= x >> 16;
    return x;
}
__host__ __device__ __forceinline__ uint32_t absorb(uint32_t h, uint32_t w) { return mix32((h ^ w) + 0x9E3779B9U); }

// per-(row, step) key of the counter-based generator; one mixing round per column follows
__host__ __device__ __forceinline__ uint32_t rowkey(uint64_t seed, uint32_t domain, uint32_t table, uint32_t row, uint64_t step) {
    uint32_t h = 0x243F6A88U;
    h = absorb(h, (uint32_t)seed); h = absorb(h, (uint32_t)(seed >> 32));
    h = absorb(h, domain); h = absorb(h, table); h = absorb(h, row);
    h = absorb(h, (uint32_t)step); h = absorb(h, (uint32_t)(step >> 32));
    return h;
}
__device__ __forceinline__ float uniform01(uint32_t key, uint32_t column) {
    uint32_t bits = mix32(key ^ (column * 0x9E3779B9U + 0x7F4A7C15U));
    return __uint2float_rn(bits >> 8) * 0x1p-24f;   // exact
}
__host__ __device__ __forceinline__ uint32_t table_salt(uint64_t seed, uint32_t table) {
    uint32_t h = 0x13198A2EU;
    h = absorb(h, (uint32_t)seed); h = absorb(h, (uint32_t)(seed >> 32)); h = absorb(h, table);
    return h;
}
// h : row -> set (Section 3 "Cache Structure")
__device__ __forceinline__ int set_of(uint32_t row, uint32_t salt, int n_sets) {
    return (int)(((uint64_t)mix32(row ^ salt) * (uint64_t)(uint32_t)n_sets) >> 32);
}

// A row of `dim` values is handled by dim/4 consecutive lanes, four columns per lane.
__device__ __forceinline__ uint32_t group_mask(int lanes_per_row) {
    const int lane = threadIdx.x & 31;
    return lanes_per_row == 32 ? 0xffffffffU : (((1U << lanes_per_row) - 1U) << (lane & ~(lanes_per_row - 1)));
}

// The four stored values of one lane (columns 4*sub .. 4*sub+3) are BITS*4 adjacent bits of the row: one byte (INT2),
// one u16 (INT4), one u32 (INT8) or two u32 (FP16 table, BITS = 16); the lowest column sits in the lowest bits.
// read-only loads of data that is used once (a low-precision row on its way to FP32): through the non-coherent path and
// without taking a line of L1, which is better spent on the FP32 rows that many bags share
__device__ __forceinline__ uint32_t ld_once_u8(const void* p) { uint32_t v; asm("ld.global.nc.L1::no_allocate.u8 %0, [%1];" : "=r"(v) : "l"(p)); return v; }
__device__ __forceinline__ uint32_t ld_once_u16(const void* p) { unsigned short v; asm("ld.global.nc.L1::no_allocate.u16 %0, [%1];" : "=h"(v) : "l"(p)); return v; }
__device__ __forceinline__ uint32_t ld_once_u32(const void* p) { uint32_t v; asm("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p)); return v; }
__device__ __forceinline__ uint2 ld_once_u32x2(const void* p) { uint2 v; asm("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p)); return v; }
__device__ __forceinline__ float2 ld_once_f32x2(const void* p) { float2 v; asm("ld.global.nc.L1::no_allocate.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "l"(p)); return v; }

template <int BITS, bool RO>
__device__ __forceinline__ uint2 load_codes4(const uint8_t* codes, int64_t grow, int dim, int sub) {
    const uint8_t* row = codes + grow * (dim * BITS / 8);
    if (BITS == 16) return RO ? ld_once_u32x2(reinterpret_cast<const uint2*>(row) + sub) : reinterpret_cast<const uint2*>(row)[sub];
    uint32_t q;
    if (BITS == 8) q = RO ? ld_once_u32(reinterpret_cast<const uint32_t*>(row) + sub) : reinterpret_cast<const uint32_t*>(row)[sub];
    else if (BITS == 4) q = RO ? ld_once_u16(reinterpret_cast<const uint16_t*>(row) + sub) : reinterpret_cast<const uint16_t*>(row)[sub];
    else q = RO ? ld_once_u8(row + sub) : row[sub];
    return make_uint2(q, 0u);
}
template <int BITS>
__device__ __forceinline__ void store_codes4(uint8_t* codes, int64_t grow, int dim, int sub, uint32_t q0, uint32_t q1, uint32_t q2, uint32_t q3) {
    uint8_t* row = codes + grow * (dim * BITS / 8);
    if (BITS == 16) { reinterpret_cast<uint2*>(row)[sub] = make_uint2(q0 | (q1 << 16), q2 | (q3 << 16)); return; }
    const uint32_t q = q0 | (q1 << (BITS & 15)) | (q2 << ((2 * BITS) & 31)) | (q3 << ((3 * BITS) & 31));
    if (BITS == 8) reinterpret_cast<uint32_t*>(row)[sub] = q;
    else if (BITS == 4) reinterpret_cast<uint16_t*>(row)[sub] = (uint16_t)q;
    else row[sub] = (uint8_t)q;
}

// Element-wise IEEE additions / fused multiply-adds, two FP32 values per instruction (the packed f32x2 forms of sm_100):
// every component is rounded to nearest exactly as the scalar instruction would round it.
__device__ __forceinline__ float4 add4(float4 a, float4 b) {
    return make_float4(__fadd_rn(a.x, b.x), __fadd_rn(a.y, b.y), __fadd_rn(a.z, b.z), __fadd_rn(a.w, b.w));
}
__device__ __forceinline__ float4 add4p(float4 a, float4 b) {
    const float2 lo = __fadd2_rn(make_float2(a.x, a.y), make_float2(b.x, b.y));
    const float2 hi = __fadd2_rn(make_float2(a.z, a.w), make_float2(b.z, b.w));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
}
__device__ __forceinline__ float4 fma4(float m, float4 g, float4 x) {       // m * g + x, fused, per component
    const float2 mm = make_float2(m, m);
    const float2 lo = __ffma2_rn(mm, make_float2(g.x, g.y), make_float2(x.x, x.y));
    const float2 hi = __ffma2_rn(mm, make_float2(g.z, g.w), make_float2(x.z, x.w));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
}
// minimum / maximum over the lanes of `mask` in one instruction (floating-point warp reduction of sm_100a)
__device__ __forceinline__ float group_min(float v, uint32_t mask) {
    float r; asm volatile("redux.sync.min.f32 %0, %1, %2;" : "=f"(r) : "f"(v), "r"(mask)); return r;
}
__device__ __forceinline__ float group_max(float v, uint32_t mask) {
    float r; asm volatile("redux.sync.max.f32 %0, %1, %2;" : "=f"(r) : "f"(v), "r"(mask)); return r;
}

// four stored values -> FP32: q*scale + bias for integer codes (Algorithm 1, up-conversion), exact for FP16
template <int BITS>
__device__ __forceinline__ float4 decode4(uint2 qq, float2 p) {
    float4 x;
    if (BITS == 16) {
        x.x = __half2float(__ushort_as_half((unsigned short)(qq.x & 0xffffu)));
        x.y = __half2float(__ushort_as_half((unsigned short)(qq.x >> 16)));
        x.z = __half2float(__ushort_as_half((unsigned short)(qq.y & 0xffffu)));
        x.w = __half2float(__ushort_as_half((unsigned short)(qq.y >> 16)));
        return x;
    }
    constexpr uint32_t M = (1u << (BITS & 15)) - 1u;
    const uint32_t q = qq.x;
    x.x = __uint2float_rn(q & M);
    x.y = __uint2float_rn((q >> (BITS & 15)) & M);
    x.z = __uint2float_rn((q >> ((2 * BITS) & 31)) & M);
    x.w = __uint2float_rn((q >> ((3 * BITS) & 31)) & M);
    return fma4(p.x, x, make_float4(p.y, p.y, p.y, p.y));      // q * s + b
}

// RO = the table is not written by the running kernel, so the read-only data path may serve the loads
template <int BITS, bool RO>
__device__ __forceinline__ float4 dequant4(const uint8_t* codes, const float2* sb, int64_t grow, int dim, int sub) {
    float2 p = make_float2(1.0f, 0.0f);
    if (BITS != 16) p = RO ? ld_once_f32x2(sb + grow) : sb[grow];
    return decode4<BITS>(load_codes4<BITS, RO>(codes, grow, dim, sub), p);
}

__device__ __forceinline__ float4 mul4(float4 a, float4 b) {
    const float2 lo = __fmul2_rn(make_float2(a.x, a.y), make_float2(b.x, b.y));
    const float2 hi = __fmul2_rn(make_float2(a.z, a.w), make_float2(b.z, b.w));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
}

// four values -> their codes; `stochastic` picks the rounding of Section 3 "Rounding" (it is the same for a whole kernel)
struct Codes4 { uint32_t q0, q1, q2, q3; };
__device__ __forceinline__ Codes4 quant4(float4 x, float mn, float inv, float qmax, uint32_t key, uint32_t column, bool stochastic) {
    // (x - b)/s as (x - b) * (1/s); x - b is formed as x + (-b), which rounds identically
    float4 y = mul4(add4p(x, make_float4(-mn, -mn, -mn, -mn)), make_float4(inv, inv, inv, inv));
    y.x = fminf(fmaxf(y.x, 0.0f), qmax); y.y = fminf(fmaxf(y.y, 0.0f), qmax);
    y.z = fminf(fmaxf(y.z, 0.0f), qmax); y.w = fminf(fmaxf(y.w, 0.0f), qmax);
    Codes4 q;
    if (stochastic) {
        const float4 f = make_float4(floorf(y.x), floorf(y.y), floorf(y.z), floorf(y.w));
        const float4 p = add4p(y, make_float4(-f.x, -f.y, -f.z, -f.w));          // y - floor(y), exact
        float4 u;                                                                // 24 random bits each, scaled to [0, 1): exact
        u.x = __uint2float_rn(mix32(key ^ (column * 0x9E3779B9U + 0x7F4A7C15U)) >> 8);
        u.y = __uint2float_rn(mix32(key ^ ((column + 1u) * 0x9E3779B9U + 0x7F4A7C15U)) >> 8);
        u.z = __uint2float_rn(mix32(key ^ ((column + 2u) * 0x9E3779B9U + 0x7F4A7C15U)) >> 8);
        u.w = __uint2float_rn(mix32(key ^ ((column + 3u) * 0x9E3779B9U + 0x7F4A7C15U)) >> 8);
        u = mul4(u, make_float4(0x1p-24f, 0x1p-24f, 0x1p-24f, 0x1p-24f));
        q.q0 = (uint32_t)f.x + (u.x < p.x ? 1u : 0u);                            // x+ with probability p: expectation y
        q.q1 = (uint32_t)f.y + (u.y < p.y ? 1u : 0u);
        q.q2 = (uint32_t)f.z + (u.z < p.z ? 1u : 0u);
        q.q3 = (uint32_t)f.w + (u.w < p.w ? 1u : 0u);
    } else {                                                                     // nearest, ties to even
        q.q0 = (uint32_t)rintf(y.x); q.q1 = (uint32_t)rintf(y.y); q.q2 = (uint32_t)rintf(y.z); q.q3 = (uint32_t)rintf(y.w);
    }
    return q;
}

// one value -> FP16 bits: the nearer neighbour, or one of the two neighbours x- <= x <= x+ (one unit in the last
// place apart) with P(x+) = (x - x-)/(x+ - x-)   (Section 3 "Rounding")
__device__ __forceinline__ uint32_t half1(float x, uint32_t key, uint32_t column, bool stochastic) {
    const float v = fminf(fmaxf(x, -65504.0f), 65504.0f);                    // stay inside the finite FP16 range
    if (!stochastic) return __half_as_ushort(__float2half_rn(v));
    const __half lo = __float2half_rd(v), hi = __float2half_ru(v);
    const unsigned short blo = __half_as_ushort(lo), bhi = __half_as_ushort(hi);
    if (blo == bhi) return blo;
    const float flo = __half2float(lo), fhi = __half2float(hi);
    const float p = __fdiv_rn(__fsub_rn(v, flo), __fsub_rn(fhi, flo));        // exact
    return uniform01(key, column) < p ? bhi : blo;
}

// Down-convert one FP32 row (four columns per lane) into the low-precision table.
template <int BITS>
__device__ __forceinline__ void quantize_store(float4 x, uint8_t* __restrict__ codes, float2* __restrict__ sb,
                                               int64_t grow, int dim, int sub, int lanes_per_row, uint32_t key, bool stochastic) {
    if (BITS == 16) {       // FP16 table: element-wise, no scale or bias
        const uint32_t c = 4u * (uint32_t)sub;
        store_codes4<BITS>(codes, grow, dim, sub, half1(x.x, key, c, stochastic), half1(x.y, key, c + 1, stochastic),
                           half1(x.z, key, c + 2, stochastic), half1(x.w, key, c + 3, stochastic));
        return;
    }
    const uint32_t mask = group_mask(lanes_per_row);
    float mn = fminf(fminf(x.x, x.y), fminf(x.z, x.w));
    float mx = fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w));
    if (lanes_per_row > 1) {                               // which zero a tie between -0 and +0 yields does not matter below
        mn = group_min(mn, mask);
        mx = group_max(mx, mask);
    }
    mn = __fadd_rn(mn, 0.0f);                              // -0 -> +0
    const float qmax = (float)((1 << (BITS & 15)) - 1);
    float s = __fdiv_rn(__fsub_rn(mx, mn), qmax);          // s = (max - min)/(2^N - 1)
    float inv = 0.0f;
    if (s >= 1.17549435e-38f) inv = __fdiv_rn(1.0f, s);
    if (inv == 0.0f) s = 0.0f;
    const uint32_t c = 4u * (uint32_t)sub;
    const Codes4 q = quant4(x, mn, inv, qmax, key, c, stochastic);
    store_codes4<BITS>(codes, grow, dim, sub, q.q0, q.q1, q.q2, q.q3);
    if (sub == 0) sb[grow] = make_float2(s, mn);
}

// ---- asynchronous 16-byte copies global -> shared (per thread; completion is waited for by group count) ----
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
// same with the shared-memory address already converted; `take` false copies nothing (the source is not read)
__device__ __forceinline__ void cp_async16_if(uint32_t smem_addr, const void* gsrc, bool take) {
    const uint32_t n = take ? 16u : 0u;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_addr), "l"(gsrc), "r"(n) : "memory");
}
// same, but the line is also kept in L1 (rows that many bags of one SM share)
__device__ __forceinline__ void cp_async16_l1(void* smem_dst, const void* gsrc) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async8(void* smem_dst, const void* gsrc) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }


}  // namespace mpe
