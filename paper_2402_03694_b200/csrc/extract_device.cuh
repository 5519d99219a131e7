// Per-flow statistical features (S1) as device code shared by the feature kernel and by the small-batch tree kernel
// that computes the features of its flows straight into its shared-memory tile.
#pragma once
#include "common.cuh"

namespace sfx {


// size groups (g0 all, g2 forward, g6 direction change): 16-bit values, at most 32 of them, so the sum fits 32 bits
struct SizeAcc { uint32_t mn, mx, s1; uint64_t s2; };
// inter-arrival groups (g1 all, g4 forward, g7 direction change): 32-bit values; sum of squares = s2a + s2b * 2^32
struct IatAcc { uint32_t mn, mx; uint64_t s1, s2a, s2b; };
// backward groups (g3 size, g5 inter-arrival): only min and max are accumulated, the sums are (all - forward)
struct MinMax { uint32_t mn, mx; };

struct Acc {
    SizeAcc z0, z2, z6;
    IatAcc a1, a4, a7;
    MinMax m3, m5;
};

__device__ __forceinline__ void acc_init(Acc& A) {
    A.z0 = A.z2 = A.z6 = SizeAcc{0xFFFFFFFFu, 0u, 0u, 0ull};
    A.a1 = A.a4 = A.a7 = IatAcc{0xFFFFFFFFu, 0u, 0ull, 0ull, 0ull};
    A.m3 = A.m5 = MinMax{0xFFFFFFFFu, 0u};
}

// c + a with a 64-bit c and a 32-bit a, written as the widening multiply-add a * 1 + c
__device__ __forceinline__ uint64_t add_wide(uint64_t c, uint32_t a) {
    uint64_t d;
    asm("mad.wide.u32 %0, %1, 1, %2;" : "=l"(d) : "r"(a), "l"(c));
    return d;
}

// Masked updates of one packet, one predicate per direction word: p = forward (bit clear) for the direction groups,
// p = direction change (bit set) for the turn groups; the updates are predicated, nothing is selected or branched.
#define SZ_UPD(P, mn, mx, s1, s2, x, sq) P " min.u32 " mn ", " mn ", " x ";\n" P " max.u32 " mx ", " mx ", " x ";\n" P " add.u32 " s1 ", " s1 ", " x ";\n" P " mad.wide.u32 " s2 ", " sq ", 1, " s2 ";\n"
#define IA_UPD(P, mn, mx, s1, s2a, s2b, x, plo, phi) P " min.u32 " mn ", " mn ", " x ";\n" P " max.u32 " mx ", " mx ", " x ";\n" P " mad.wide.u32 " s1 ", " x ", 1, " s1 ";\n" P " mad.wide.u32 " s2a ", " plo ", 1, " s2a ";\n" P " mad.wide.u32 " s2b ", " phi ", 1, " s2b ";\n"
#define MM_UPD(P, mn, mx, x) P " min.u32 " mn ", " mn ", " x ";\n" P " max.u32 " mx ", " mx ", " x ";\n"
#define PRED_EQ(word, bit) "{\n.reg .pred p;\n.reg .b32 t;\nand.b32 t, " word ", " bit ";\nsetp.eq.u32 p, t, 0;\n"
#define PRED_NE(word, bit) "{\n.reg .pred p;\n.reg .b32 t;\nand.b32 t, " word ", " bit ";\nsetp.ne.u32 p, t, 0;\n"

template <int G>
__device__ __forceinline__ void dir_groups(Acc& A, uint32_t sz, uint32_t sq, uint32_t ia, uint32_t plo, uint32_t phi, uint32_t dirw, uint32_t bit) {
    if (G >= 6)
        asm(PRED_EQ("%18", "%19") SZ_UPD("@p", "%0", "%1", "%2", "%3", "%13", "%14") MM_UPD("@!p", "%4", "%5", "%13")
            IA_UPD("@p", "%6", "%7", "%8", "%9", "%10", "%15", "%16", "%17") MM_UPD("@!p", "%11", "%12", "%15") "}"
            : "+r"(A.z2.mn), "+r"(A.z2.mx), "+r"(A.z2.s1), "+l"(A.z2.s2), "+r"(A.m3.mn), "+r"(A.m3.mx), "+r"(A.a4.mn), "+r"(A.a4.mx),
              "+l"(A.a4.s1), "+l"(A.a4.s2a), "+l"(A.a4.s2b), "+r"(A.m5.mn), "+r"(A.m5.mx)
            : "r"(sz), "r"(sq), "r"(ia), "r"(plo), "r"(phi), "r"(dirw), "r"(bit));
    else if (G == 5)
        asm(PRED_EQ("%16", "%17") SZ_UPD("@p", "%0", "%1", "%2", "%3", "%11", "%12") MM_UPD("@!p", "%4", "%5", "%11")
            IA_UPD("@p", "%6", "%7", "%8", "%9", "%10", "%13", "%14", "%15") "}"
            : "+r"(A.z2.mn), "+r"(A.z2.mx), "+r"(A.z2.s1), "+l"(A.z2.s2), "+r"(A.m3.mn), "+r"(A.m3.mx), "+r"(A.a4.mn), "+r"(A.a4.mx),
              "+l"(A.a4.s1), "+l"(A.a4.s2a), "+l"(A.a4.s2b)
            : "r"(sz), "r"(sq), "r"(ia), "r"(plo), "r"(phi), "r"(dirw), "r"(bit));
    else if (G == 4)
        asm(PRED_EQ("%8", "%9") SZ_UPD("@p", "%0", "%1", "%2", "%3", "%6", "%7") MM_UPD("@!p", "%4", "%5", "%6") "}"
            : "+r"(A.z2.mn), "+r"(A.z2.mx), "+r"(A.z2.s1), "+l"(A.z2.s2), "+r"(A.m3.mn), "+r"(A.m3.mx)
            : "r"(sz), "r"(sq), "r"(dirw), "r"(bit));
    else if (G == 3)
        asm(PRED_EQ("%6", "%7") SZ_UPD("@p", "%0", "%1", "%2", "%3", "%4", "%5") "}"
            : "+r"(A.z2.mn), "+r"(A.z2.mx), "+r"(A.z2.s1), "+l"(A.z2.s2)
            : "r"(sz), "r"(sq), "r"(dirw), "r"(bit));
}
template <int G>
__device__ __forceinline__ void turn_groups(Acc& A, uint32_t sz, uint32_t sq, uint32_t ia, uint32_t plo, uint32_t phi, uint32_t turnw, uint32_t bit) {
    if (G >= 8)
        asm(PRED_NE("%14", "%15") SZ_UPD("@p", "%0", "%1", "%2", "%3", "%9", "%10") IA_UPD("@p", "%4", "%5", "%6", "%7", "%8", "%11", "%12", "%13") "}"
            : "+r"(A.z6.mn), "+r"(A.z6.mx), "+r"(A.z6.s1), "+l"(A.z6.s2), "+r"(A.a7.mn), "+r"(A.a7.mx), "+l"(A.a7.s1), "+l"(A.a7.s2a), "+l"(A.a7.s2b)
            : "r"(sz), "r"(sq), "r"(ia), "r"(plo), "r"(phi), "r"(turnw), "r"(bit));
    else if (G == 7)
        asm(PRED_NE("%6", "%7") SZ_UPD("@p", "%0", "%1", "%2", "%3", "%4", "%5") "}"
            : "+r"(A.z6.mn), "+r"(A.z6.mx), "+r"(A.z6.s1), "+l"(A.z6.s2)
            : "r"(sz), "r"(sq), "r"(turnw), "r"(bit));
}
#undef SZ_UPD
#undef IA_UPD
#undef MM_UPD
#undef PRED_EQ
#undef PRED_NE

// One packet of the window.  Groups: g0 size/all, g1 iat/all, g2 size/fwd, g3 size/bwd, g4 iat/fwd, g5 iat/bwd,
// g6 size/turn, g7 iat/turn.  dirw: bit set = backward packet; turnw: bit set = direction differs from the packet before.
template <int G>
__device__ __forceinline__ void packet(Acc& A, uint32_t sz, uint32_t ia, uint32_t dirw, uint32_t turnw, uint32_t bit) {
    const uint32_t sq = sz * sz;                                  // 16-bit sizes: the square fits 32 bits
    A.z0.mn = min(A.z0.mn, sz); A.z0.mx = max(A.z0.mx, sz); A.z0.s1 += sz; A.z0.s2 = add_wide(A.z0.s2, sq);
    uint32_t plo = 0, phi = 0;
    if (G > 1) {
        const uint64_t p = (uint64_t)ia * (uint64_t)ia;
        plo = (uint32_t)p; phi = (uint32_t)(p >> 32);
        A.a1.mn = min(A.a1.mn, ia); A.a1.mx = max(A.a1.mx, ia);
        A.a1.s1 = add_wide(A.a1.s1, ia); A.a1.s2a = add_wide(A.a1.s2a, plo); A.a1.s2b = add_wide(A.a1.s2b, phi);
    }
    if (G > 2) dir_groups<G>(A, sz, sq, ia, plo, phi, dirw, bit);
    if (G > 6) turn_groups<G>(A, sz, sq, ia, plo, phi, turnw, bit);
}

// exact unsigned 128-bit value (hi:lo) -> fp32, round to nearest even.
// Above 64 bits: normalise into a 64-bit window, OR the dropped bits into a
// sticky bit (it sits far below the rounding position), convert once, and scale
// by an exact power of two.
__device__ __forceinline__ float u128_to_f32(uint64_t hi, uint64_t lo) {
    if (hi == 0) return __ull2float_rn(lo);
    int s = 64 - __clzll((long long)hi);                     // 1..64
    uint64_t w = (s == 64) ? hi : ((hi << (64 - s)) | (lo >> s));
    uint64_t dropped = (s == 64) ? lo : (lo << (64 - s));
    w |= (dropped != 0) ? 1ull : 0ull;
    float f = __ull2float_rn(w);
    return __fmul_rn(f, __uint_as_float((uint32_t)(127 + s) << 23));   // * 2^s, exact
}

// Where a flow's features go.  RowOut: a row of 8 * G floats (16-byte aligned; two 16-byte stores per group).
// ColOut: column `col` of a transposed tile xs[feature][stride] (the tree kernels' layout).
struct RowOut {
    float* o;
    __device__ __forceinline__ void put(int g, float4 lo, float4 hi) const {
        float4* o4 = reinterpret_cast<float4*>(o + 8 * g);       // conflict-free across a quarter warp
        o4[0] = lo; o4[1] = hi;
    }
};
struct ColOut {
    float* xs; uint32_t stride;
    __device__ __forceinline__ void put(int g, float4 lo, float4 hi) const {
        float* c = xs + (size_t)(8 * g) * stride;
        c[0] = lo.x; c[stride] = lo.y; c[2 * stride] = lo.z; c[3 * stride] = lo.w;
        c[4 * stride] = hi.x; c[5 * stride] = hi.y; c[6 * stride] = hi.z; c[7 * stride] = hi.w;
    }
};

// eight slots of one group: cnt, sum, min, max, mean, var, first, last
template <typename Out>
__device__ __forceinline__ void store_slots(const Out& out, int g, float fc, float fs, uint32_t mn, uint32_t mx, float fv, uint32_t cnt,
                                            uint32_t first, uint32_t last) {
    out.put(g, make_float4(fc, fs, __uint2float_rn(mn), __uint2float_rn(mx)),
            make_float4(__fdiv_rn(fs, fc), __fdiv_rn(fv, __uint2float_rn(cnt * cnt)), __uint2float_rn(first), __uint2float_rn(last)));
}
template <typename Out>
__device__ __forceinline__ void store_empty(const Out& out, int g) {
    out.put(g, make_float4(0.0f, 0.0f, 0.0f, 0.0f), make_float4(0.0f, 0.0f, 0.0f, 0.0f));
}
// size group: S1 < 2^21 and cnt * S2, S1^2 < 2^42, so the variance numerator V = cnt * S2 - S1^2 is a 64-bit integer
template <typename Out>
__device__ __forceinline__ void finish_size(uint32_t cnt, uint32_t mn, uint32_t mx, uint32_t s1, uint64_t s2,
                                            uint32_t first, uint32_t last, const Out& o, int g) {
    if (cnt == 0) { store_empty(o, g); return; }
    const uint64_t v = (uint64_t)cnt * s2 - (uint64_t)s1 * (uint64_t)s1;
    store_slots(o, g, __uint2float_rn(cnt), __uint2float_rn(s1), mn, mx, __ull2float_rn(v), cnt, first, last);
}
// inter-arrival group: S2 = s2a + s2b * 2^32 (up to 2^69), V = cnt * S2 - S1^2 as an exact 128-bit integer
template <typename Out>
__device__ __forceinline__ void finish_iat(uint32_t cnt, uint32_t mn, uint32_t mx, uint64_t s1, uint64_t s2a, uint64_t s2b,
                                           uint32_t first, uint32_t last, const Out& o, int g) {
    if (cnt == 0) { store_empty(o, g); return; }
    const uint64_t s2lo = s2a + (s2b << 32);
    const uint64_t s2hi = (s2b >> 32) + ((s2lo < s2a) ? 1ull : 0ull);
    const uint64_t c = cnt;
    const uint64_t p_lo = c * s2lo;
    const uint64_t p_hi = __umul64hi(c, s2lo) + c * s2hi;
    const uint64_t q_lo = s1 * s1;
    const uint64_t q_hi = __umul64hi(s1, s1);
    const uint64_t v_lo = p_lo - q_lo;
    const uint64_t v_hi = p_hi - q_hi - ((p_lo < q_lo) ? 1ull : 0ull);
    store_slots(o, g, __uint2float_rn(cnt), __ull2float_rn(s1), mn, mx, u128_to_f32(v_hi, v_lo), cnt, first, last);
}

// All 8 * G features of one flow whose packets are row `fr` of the planes (pitch packets per row); m = packets in the
// window (at most N <= 32, so all direction bits of the window are in the row's first word, dirw).
template <int G, bool VEC, typename Out>
__device__ __forceinline__ void extract_flow(const uint16_t* __restrict__ size, const uint32_t* __restrict__ iat, size_t fr, uint32_t pitch,
                                         uint32_t m, uint32_t dirw, const Out& out)
{
    Acc A;
    acc_init(A);
    const uint32_t turnw = (dirw ^ (dirw << 1)) & ~1u;        // packet i >= 1 whose direction differs from i-1
    const uint32_t all_mask = (m >= 32) ? 0xFFFFFFFFu : ((1u << m) - 1u);
    const uint16_t* srow = size + fr * pitch;
    const uint32_t* irow = iat + fr * pitch;
    uint32_t done = 0;                             // packets accumulated so far
    if (VEC) {
        const uint32_t n_full = m >> 3;
        uint4 s4, a4, b4;
        if (n_full) {
            s4 = __ldg(reinterpret_cast<const uint4*>(srow)); a4 = __ldg(reinterpret_cast<const uint4*>(irow));
            b4 = __ldg(reinterpret_cast<const uint4*>(irow + 4));
        }
#pragma unroll 1
        for (uint32_t ch = 0; ch < n_full; ch++) {
            const uint4 cs = s4, ca = a4, cb = b4;
            if (ch + 1 < n_full) {
                s4 = __ldg(reinterpret_cast<const uint4*>(srow + (ch + 1) * 8)); a4 = __ldg(reinterpret_cast<const uint4*>(irow + (ch + 1) * 8));
                b4 = __ldg(reinterpret_cast<const uint4*>(irow + (ch + 1) * 8 + 4));
            }
            const uint32_t sz[8] = {cs.x & 0xFFFFu, cs.x >> 16, cs.y & 0xFFFFu, cs.y >> 16, cs.z & 0xFFFFu, cs.z >> 16, cs.w & 0xFFFFu, cs.w >> 16};
            const uint32_t ia[8] = {ca.x, ca.y, ca.z, ca.w, cb.x, cb.y, cb.z, cb.w};
            const uint32_t dw = dirw >> (8 * ch), tw = turnw >> (8 * ch);
#pragma unroll
            for (int j = 0; j < 8; j++) packet<G>(A, sz[j], ia[j], dw, tw, 1u << j);
        }
        done = n_full * 8;
    }
    for (uint32_t i = done; i < m; i++) packet<G>(A, srow[i], irow[i], dirw, turnw, 1u << i);      // ragged end / unaligned rows

    const uint32_t fwd_mask = ~dirw & all_mask, bwd_mask = dirw & all_mask, turn_mask = turnw & all_mask;
#pragma unroll
    for (int g = 0; g < G; g++) {
        const uint32_t mask = (g < 2) ? all_mask : (g == 2 || g == 4) ? fwd_mask : (g == 3 || g == 5) ? bwd_mask : turn_mask;
        const bool is_size = (g == 0 || g == 2 || g == 3 || g == 6);
        const uint32_t cnt = __popc(mask);
        uint32_t first = 0, last = 0;
        if (cnt) {                               // the row was just read: these hit in L1
            const uint32_t i0 = __ffs(mask) - 1, i1 = 31 - __clz(mask);
            first = is_size ? (uint32_t)srow[i0] : irow[i0];
            last = is_size ? (uint32_t)srow[i1] : irow[i1];
        }
        if (g == 0) finish_size(cnt, A.z0.mn, A.z0.mx, A.z0.s1, A.z0.s2, first, last, out, g);
        else if (g == 1) finish_iat(cnt, A.a1.mn, A.a1.mx, A.a1.s1, A.a1.s2a, A.a1.s2b, first, last, out, g);
        else if (g == 2) finish_size(cnt, A.z2.mn, A.z2.mx, A.z2.s1, A.z2.s2, first, last, out, g);
        else if (g == 3) finish_size(cnt, A.m3.mn, A.m3.mx, A.z0.s1 - A.z2.s1, A.z0.s2 - A.z2.s2, first, last, out, g);
        else if (g == 4) finish_iat(cnt, A.a4.mn, A.a4.mx, A.a4.s1, A.a4.s2a, A.a4.s2b, first, last, out, g);
        else if (g == 5) finish_iat(cnt, A.m5.mn, A.m5.mx, A.a1.s1 - A.a4.s1, A.a1.s2a - A.a4.s2a, A.a1.s2b - A.a4.s2b, first, last, out, g);
        else if (g == 6) finish_size(cnt, A.z6.mn, A.z6.mx, A.z6.s1, A.z6.s2, first, last, out, g);
        else finish_iat(cnt, A.a7.mn, A.a7.mx, A.a7.s1, A.a7.s2a, A.a7.s2b, first, last, out, g);
    }
}

}  // namespace sfx
