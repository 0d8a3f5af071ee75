// Brute-force scale search (Experimental Setup: the optimal baseline, found by trying the possible
// scale values and keeping the one with the least error): every finite scale code of the format
// is tried on every block and the code with the smallest SSE is kept (equal SSE: the smaller code).
//
// Work layout.  A thread keeps its elements in registers as float pairs and the candidate loop
// works on float pairs with the packed binary32 instructions of sm_100 (fma.rn.f32x2 /
// mul.rn.f32x2, FP4 pack and unpack two at a time):
//   B <= 16   the thread owns G = 32 consecutive elements (16 for B = 2), pair i = (element i,
//             element G/2 + i): the two halves of a pair belong to different blocks, so one instruction serves two
//             elements of one candidate and the two SSE chains are independent.  Two candidates
//             per trip.
//   B >= 32   the thread owns one block, pair i = (element 2i, element 2i + 1).  Its SSE is one
//             sequential chain over all elements, so the two lanes of the SSE pair are two
//             CANDIDATES: the scaling multiplies run on element pairs, the FP4 rounding and the
//             residuals on candidate pairs of one element, and the elements are walked in order.
// The candidate loop is uniform across the CTA: decode scales come from shared memory as
// broadcasts.
//
// One exact quotient per mantissa, not per candidate.  The decode scale of code c is
// D_c = fl(S_c * g).  All codes whose S_c share a mantissa (eight classes for the FP8 scale
// formats, one for the power-of-two format) have decode scales that differ by exact powers of two,
// D_c = Dref * 2^k, as long as D_c is a normal number.  Hence fl(v / D_c) = fl(v / Dref) * 2^-k
// exactly: the correctly rounded quotient is formed once per class and element, and a candidate
// costs one multiply by a power of two, the FP4 rounding, and the two FMAs of the SSE.  Codes
// whose decode scale is zero, subnormal or above 2^126 need no quotient at all (every element
// rounds to zero, or saturates) and form one more list.  Threads holding a magnitude above 2^60
// or a nonzero one below 2^-62 take the general path (IEEE division), candidate by candidate.
//
// Inside a class the members are visited in ascending code order and the smallest SSE bit pattern
// is kept with a strict compare (SSE >= 0, so integer order is float order and the first of equals
// is the smaller code); class winners are merged as 64-bit keys (SSE bits << 32 | code).
#pragma once

#include <atomic>

#include "mxq_device.cuh"
#include "mxq_internal.h"

namespace mxq {

constexpr int kMaxMembers = 36;  // codes per mantissa class, FP8 formats (31 normal + 3 subnormal at most)

// Mantissa class of a scale code: index of the 3-bit mantissa of its value.
template <int FMT>
__device__ __forceinline__ int code_class(int c) {
    if constexpr (FMT == kUE8M0) return 0;
    if (c >= 8) return c & 7;
    // subnormal codes m * 2^(1-bias-3): 1, 2, 4 -> 1.0; 3, 6 -> 1.5; 5 -> 1.25; 7 -> 1.75
    return (int)((0x64204000u >> (4 * c)) & 7u);
}

// Per-CTA tables of the search.  Every code with a finite decode scale D sits in one candidate list:
//   * D normal with a biased exponent of at most 253 ("paired": D = Dref * 2^k and 2^-k are both
//     representable): list 2 * class + kind, where kind 1 holds the codes whose -D is exactly
//     representable in f16 (their residual is one mixed-precision FMA from the unpacked f16 grid
//     value) and kind 0 the others (f16 -> f32 convert, then an FFMA);
//   * the "flat" list kFlatList for the rest.  D = 0 or D >= 2^127: every quotient of a magnitude
//     <= 2^60 rounds to FP4 zero, so the candidate is entered with the multiplier 0.  D subnormal:
//     every nonzero magnitude >= 2^-62 divided by it exceeds 2^64 and saturates at 6, so it is
//     entered with the multiplier 2^126.  The flat list is evaluated on the elements themselves
//     (Dref = 1), which needs no quotient.
constexpr int kLists = 17;
constexpr int kFlatList = 16;
constexpr int kCandSlots = 16 * kMaxMembers + 256;
struct BruteTables {
    float D[256];            // decode scale of the code; NaN for codes that do not exist
    float R[256];            // RN(1 / D) when 2^-60 <= D <= 2^60, else 0 (used by the final encode)
    float4 cand[kCandSlots];    // per list, ascending code order: (-D, multiplier, f16(-D) twice as bits, 0)
    uint8_t member[kCandSlots]; // the code of each slot of cand[]
    uint8_t kind[256];       // 0, 1 paired as above; 3 = flat list; 2 = not a candidate
    float clsD[8];           // Dref of the class, in [1, 2)
    float clsR[8];           // RN(1 / Dref)
    int cnt[kLists];         // members per list
    uint32_t kind_mask[3][8];
    // pruned sweep only
    uint8_t below[kLists - 1][256];  // below[list][E]: members of the paired list whose D has a biased exponent < E
    int flat_zero_min;               // smallest code of the flat list that has the multiplier 0; 256 if none
};

template <int FMT>
__device__ __forceinline__ int members_base(int list) {
    if (list == kFlatList) return 16 * kMaxMembers;
    // the power-of-two format has one class: its two lists get half of the class area each
    return FMT == kUE8M0 ? list * (16 * kMaxMembers / 2) : list * kMaxMembers;
}

// first: smallest admissible code (1 under prevent-zero for the FP8 formats, else 0).
// PRUNE: also the exponent index of the lists that the pruned sweep cuts its ranges with.
template <int FMT, bool PRUNE>
__device__ __forceinline__ void build_brute_tables(BruteTables& T, float g, int first) {
    static_assert(kThreads == 256, "one thread per table entry");
    build_scale_tables<FMT>(T.D, T.R, g);
    const int c = threadIdx.x;
    const float D = T.D[c];
    const uint32_t b = __float_as_uint(D);
    const uint32_t e = (b >> 23) & 0xFFu;
    const bool usable = c >= first && c < num_codes(FMT) && (b >> 31) == 0 && e != 255;
    const bool is_paired = usable && e >= 1 && e <= 253;
    const __half hD = __float2half_rn(-D);
    const int kind = !usable ? 2 : (!is_paired ? 3 : (__half2float(hD) == -D ? 1 : 0));
    T.kind[c] = (uint8_t)kind;
    if (c < kLists) T.cnt[c] = 0;
    if (c == 0) T.flat_zero_min = 256;
    const uint32_t ballot0 = __ballot_sync(0xFFFFFFFFu, kind == 0);
    const uint32_t ballot1 = __ballot_sync(0xFFFFFFFFu, kind == 1);
    const uint32_t ballot3 = __ballot_sync(0xFFFFFFFFu, kind == 3);
    if ((c & 31) == 0) {
        T.kind_mask[0][c >> 5] = ballot0;
        T.kind_mask[1][c >> 5] = ballot1;
        T.kind_mask[2][c >> 5] = ballot3;
    }
    __syncthreads();
    const uint32_t below = (1u << (c & 31)) - 1u;
    if (kind == 3) {
        int rank = __popc(ballot3 & below);
        for (int w = 0; w < (c >> 5); ++w) rank += __popc(T.kind_mask[2][w]);
        // multiplier 0 -> every quotient is zero; 2^126 -> every nonzero quotient saturates
        const float P = (e == 0 && D != 0.0f) ? __uint_as_float(0x7E800000u) : 0.0f;
        const int slot = members_base<FMT>(kFlatList) + rank;
        T.cand[slot] = make_float4(-D, P, 0.0f, 0.0f);
        T.member[slot] = (uint8_t)c;
        atomicAdd(&T.cnt[kFlatList], 1);
        if (P == 0.0f) atomicMin(&T.flat_zero_min, c);
    }
    int my_list = -1, my_rank = 0;
    if (is_paired) {
        const int cls = code_class<FMT>(c);
        int rank = 0;
        if constexpr (FMT == kUE8M0) {
            for (int w = 0; w < (c >> 5); ++w) rank += __popc(T.kind_mask[kind][w]);
            rank += __popc((kind ? ballot1 : ballot0) & below);
        } else {
            for (int o = 1; o < 8 && o < c; ++o) rank += (T.kind[o] == kind && code_class<FMT>(o) == cls) ? 1 : 0;
            for (int o = 8 + cls; o < c; o += 8) rank += (T.kind[o] == kind) ? 1 : 0;
        }
        const float P = __uint_as_float((254u - e) << 23);
        const uint32_t h16 = (uint32_t)__half_as_ushort(hD);
        const int list = 2 * cls + kind;
        const int slot = members_base<FMT>(list) + rank;
        T.cand[slot] = make_float4(-D, P, __uint_as_float(h16 | (h16 << 16)), 0.0f);
        T.member[slot] = (uint8_t)c;
        atomicAdd(&T.cnt[list], 1);
        my_list = list;
        my_rank = rank;
        if (rank == 0) {   // both kinds of a class write the same values
            const float Dref = __uint_as_float((b & 0x007FFFFFu) | 0x3F800000u);
            T.clsD[cls] = Dref;
            T.clsR[cls] = __frcp_rn(Dref);
        }
    }
    __syncthreads();
    // the search takes two members per trip: a range that ends with the list may read one slot
    // past it, which repeats the last member
    if (c < kLists && T.cnt[c] > 0) {
        const int last = members_base<FMT>(c) + T.cnt[c] - 1;
        T.cand[last + 1] = T.cand[last];
        T.member[last + 1] = T.member[last];
    }
    if constexpr (PRUNE) {
        // Exponents rise strictly along a paired list (one member per binade of its class), so
        // member `rank` owns the exponents above its predecessor's up to its own, and the last
        // member also those above.
        if (my_list >= 0) {
            const int slot = members_base<FMT>(my_list) + my_rank;
            const int e_prev = my_rank > 0 ? (int)((__float_as_uint(T.cand[slot - 1].x) >> 23) & 0xFFu) : -1;
            for (int E = e_prev + 1; E <= (int)e; ++E) T.below[my_list][E] = (uint8_t)my_rank;
            if (my_rank == T.cnt[my_list] - 1)
                for (int E = (int)e + 1; E < 256; ++E) T.below[my_list][E] = (uint8_t)(my_rank + 1);
        }
        for (int l = 0; l < kLists - 1; ++l)
            if (T.cnt[l] == 0) T.below[l][c] = 0;
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------------------------
// packed helpers
// ------------------------------------------------------------------------------------------------
// Residuals of one pair for one candidate: t = tb * 2^-k, q = t rounded onto the FP4 grid
// (round-to-nearest-even, saturating at +-6), e = fma(q, -D, v).  HALF: -D is given in f16
// (low half of nD16 for .x, high half for .y) and the FMA takes q straight from the unpacked f16
// pair (fma.rn.f32.f16: exact product, one rounding to binary32); otherwise q is widened first.
template <bool HALF>
__device__ __forceinline__ float2 residual_pair(float2 tb, float2 P2, float2 v, float2 nD2, uint32_t nD16) {
    const float2 t = __fmul2_rn(tb, P2);
    uint32_t h;
    asm("{\n"
        " .reg .b8 b0;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n"
        " cvt.rn.f16x2.e2m1x2 %0, b0;\n"
        "}"
        : "=r"(h)
        : "f"(t.x), "f"(t.y));
    if constexpr (HALF) {
        float2 e;
        asm("{\n"
            " .reg .b16 qlo, qhi, dlo, dhi;\n"
            " mov.b32 {qlo, qhi}, %2;\n"
            " mov.b32 {dlo, dhi}, %3;\n"
            " fma.rn.f32.f16 %0, qlo, dlo, %4;\n"
            " fma.rn.f32.f16 %1, qhi, dhi, %5;\n"
            "}"
            : "=f"(e.x), "=f"(e.y)
            : "r"(h), "r"(nD16), "f"(v.x), "f"(v.y));
        return e;
    } else {
        // f16 -> binary32 as a mixed-precision add of -0 (exact, keeps the sign of zero): unlike a
        // plain convert it takes its half straight out of the 32-bit register
        float2 q;
        asm("{\n"
            " .reg .b16 qlo, qhi;\n"
            " mov.b32 {qlo, qhi}, %2;\n"
            " add.rn.f32.f16 %0, qlo, %3;\n"
            " add.rn.f32.f16 %1, qhi, %3;\n"
            "}"
            : "=f"(q.x), "=f"(q.y)
            : "r"(h), "f"(-0.0f));
        return make_float2(__fmaf_rn(q.x, nD2.x, v.x), __fmaf_rn(q.y, nD2.y, v.y));
    }
}

// Residuals of ONE element for TWO candidates A, B, given its scaled quotients tA = tb * 2^-kA and
// tB: q = FP4 rounding of t, e = fma(q, -D, v) for either candidate (.x = A, .y = B).  HALF: nD16
// holds f16(-D_A) in the low half and f16(-D_B) in the high half.
template <bool HALF>
__device__ __forceinline__ float2 residual_two_candidates(float tA, float tB, float v, float nDA, float nDB,
                                                          uint32_t nD16) {
    uint32_t h;
    asm("{\n"
        " .reg .b8 b0;\n"
        " cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n"
        " cvt.rn.f16x2.e2m1x2 %0, b0;\n"
        "}"
        : "=r"(h)
        : "f"(tA), "f"(tB));
    float2 e;
    if constexpr (HALF) {
        asm("{\n"
            " .reg .b16 qlo, qhi, dlo, dhi;\n"
            " mov.b32 {qlo, qhi}, %2;\n"
            " mov.b32 {dlo, dhi}, %3;\n"
            " fma.rn.f32.f16 %0, qlo, dlo, %4;\n"
            " fma.rn.f32.f16 %1, qhi, dhi, %4;\n"
            "}"
            : "=f"(e.x), "=f"(e.y)
            : "r"(h), "r"(nD16), "f"(v));
    } else {
        float2 q;   // f16 -> binary32 as in residual_pair()
        asm("{\n"
            " .reg .b16 qlo, qhi;\n"
            " mov.b32 {qlo, qhi}, %2;\n"
            " add.rn.f32.f16 %0, qlo, %3;\n"
            " add.rn.f32.f16 %1, qhi, %3;\n"
            "}"
            : "=f"(q.x), "=f"(q.y)
            : "r"(h), "f"(-0.0f));
        e.x = __fmaf_rn(q.x, nDA, v);
        e.y = __fmaf_rn(q.y, nDB, v);
    }
    return e;
}

// fl32(v / Dref) for both halves; nD = -Dref, R = RN(1 / Dref), Dref in [1, 2), |v| <= 2^60: the
// reciprocal multiply with one residual correction of quotient_short() (see there why one
// correction gives the IEEE quotient for every divisor), except for the sign of a zero quotient,
// which the search does not use.
__device__ __forceinline__ float2 quotient_pair(float2 v, float2 nD, float2 R) {
    const float2 q = __fmul2_rn(v, R);
    const float2 r = __ffma2_rn(q, nD, v);
    return __ffma2_rn(r, R, q);
}

__device__ __forceinline__ unsigned long long sse_key(float s, int c) {
    return ((unsigned long long)__float_as_uint(s) << 32) | (unsigned long long)(unsigned)c;
}

// General path for one block held in `lane` (0 = .x, 1 = .y) of pairs first .. first + B - 1.
template <int B, int NP>
__device__ __forceinline__ float general_sse(const float2 (&v2)[NP], int first, int lane, float D) {
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < B; i += 2) {
        const float a = lane ? v2[first + i].y : v2[first + i].x;
        const float b = lane ? v2[first + i + 1].y : v2[first + i + 1].x;
        const float2 q = round_e2m1x2(quotient_general(a, D), quotient_general(b, D));
        const float e0 = __fmaf_rn(-q.x, D, a);
        s = __fmaf_rn(e0, e0, s);
        const float e1 = __fmaf_rn(-q.y, D, b);
        s = __fmaf_rn(e1, e1, s);
    }
    return s;
}

// ------------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------------
// Fold the winner of one class (smallest SSE bits; first, i.e. smallest, code among equals) into
// the running (SSE, code) key.
__device__ __forceinline__ void merge_class_winner(unsigned long long& best, uint32_t bits, int code) {
    const unsigned long long k = ((unsigned long long)bits << 32) | (unsigned long long)(unsigned)code;
    if (k < best) best = k;
}

// Strict "smaller SSE bits wins", without a branch.
__device__ __forceinline__ void keep_smaller(uint32_t& best_bits, int& best_slot, uint32_t bits, int slot) {
    best_slot = bits < best_bits ? slot : best_slot;
    best_bits = min(best_bits, bits);
}

// ------------------------------------------------------------------------------------------------
// Pruned sweep.  Three facts about a candidate D let a warp leave it out without changing any
// output (they concern the thread's elements v, magnitudes a = max |v| of a block, and the SSE as
// the kernel computes it: e = fma(q, -D, v), s = fma(e, e, s) in element order; binary32 rounding
// is monotone, so a sum of squares never decreases when a term is added or a term grows):
//   zero rule   D >= 4 * (largest magnitude in the warp): every quotient is at most 1/4 and rounds
//               to the grid value 0 (the tie goes to the even index), so every such candidate has
//               exactly the SSE of the all-zero quantization.  That SSE is entered once, with the
//               smallest such code.
//   high rule   D >= 4 * theta: the elements with |v| <= theta quantize to zero, so the SSE of a
//               block is at least Z = the sum of squares of those elements (same order).  If
//               Z > best SSE found so far, for every block of the warp, no such candidate can win
//               or tie.  theta = largest magnitude * 2^-j, j = 2, 3, 4.
//   low rule    6 * D <= a: the largest element saturates at 6 and leaves the error
//               e = fl(a - 6 D), so the SSE is at least fl(e * e).  Every D below a D' that passes
//               "fl(fl(a - 6 D')^2) > best SSE so far" (smallest a and largest best SSE of the
//               thread's blocks; then the smallest D' of the warp) can neither win nor tie.
// The cuts are taken per mantissa class from the exponent index below[][]: D = Dref * 2^E is
// below a limit L = mL * 2^eL  <=>  E < eL + (Dref < mL).
// ------------------------------------------------------------------------------------------------
// Exponent cut of a limit (bit pattern of a non-negative binary32, +inf allowed) for a class whose
// reference has the significand field cls_mant: the members of the class's lists with a biased
// exponent below the cut, T.below[list][cut] of them, are the ones whose decode scale is below
// the limit.
__device__ __forceinline__ uint32_t exponent_cut(uint32_t cls_mant, uint32_t limit_bits) {
    const uint32_t eL = limit_bits >> 23, mL = limit_bits & 0x007FFFFFu;
    return min(eL + (cls_mant < mL ? 1u : 0u), 255u);
}

// limit * 2^-j for a limit given as bits (0 when that leaves the normal range)
__device__ __forceinline__ uint32_t limit_shifted_down(uint32_t limit_bits, int j) {
    return (limit_bits >> 23) > (uint32_t)j ? limit_bits - ((uint32_t)j << 23) : 0u;
}

// All members of one range of one list (one mantissa class, one residual kind) against the
// thread's elements; the winner of every block is folded into best[].
// Members first .. first + cnt_raw - 1 of the list are evaluated.
template <int B, int FMT, bool HALF, int NP, int NBT>
__device__ __forceinline__ void search_list(const BruteTables& T, int list, int first, int cnt_raw,
                                            const float2 (&v2)[NP], const float2 (&tb)[NP],
                                            unsigned long long (&best)[NBT]) {
    constexpr bool ONEBLK = (B >= 32);
    constexpr int BL = ONEBLK ? NP : B;
    constexpr int NBL = NP / BL;
    if (cnt_raw <= 0) return;
    [[maybe_unused]] const int cnt = cnt_raw;
    const int base = members_base<FMT>(list) + first;
    const float4* cand = T.cand + base;
    uint32_t cbest[NBT];
    int cslot[NBT];
#pragma unroll
    for (int k = 0; k < NBT; ++k) { cbest[k] = 0xFFFFFFFFu; cslot[k] = 0; }

    if constexpr (!ONEBLK) {
        // two members per trip: two independent SSE chains keep the FMA pipe fed
        const int pairs_end = cnt & ~1;
        for (int m = 0; m < pairs_end; m += 2) {
            const float4 dpA = cand[m], dpB = cand[m + 1];
            const float2 nDA = make_float2(dpA.x, dpA.x), PA = make_float2(dpA.y, dpA.y);
            const float2 nDB = make_float2(dpB.x, dpB.x), PB = make_float2(dpB.y, dpB.y);
            const uint32_t hA = __float_as_uint(dpA.z), hB = __float_as_uint(dpB.z);
            float2 sA[NBL], sB[NBL];
#pragma unroll
            for (int k = 0; k < NBL; ++k) sA[k] = sB[k] = make_float2(0.0f, 0.0f);
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                const float2 eA = residual_pair<HALF>(tb[i], PA, v2[i], nDA, hA);
                const float2 eB = residual_pair<HALF>(tb[i], PB, v2[i], nDB, hB);
                sA[i / BL] = __ffma2_rn(eA, eA, sA[i / BL]);
                sB[i / BL] = __ffma2_rn(eB, eB, sB[i / BL]);
            }
#pragma unroll
            for (int k = 0; k < NBL; ++k) {
                keep_smaller(cbest[k], cslot[k], __float_as_uint(sA[k].x), m);
                keep_smaller(cbest[NBL + k], cslot[NBL + k], __float_as_uint(sA[k].y), m);
                keep_smaller(cbest[k], cslot[k], __float_as_uint(sB[k].x), m + 1);
                keep_smaller(cbest[NBL + k], cslot[NBL + k], __float_as_uint(sB[k].y), m + 1);
            }
        }
        if (cnt & 1) {   // the odd member on its own
            const int m = cnt - 1;
            const float4 dpA = cand[m];
            const float2 nDA = make_float2(dpA.x, dpA.x), PA = make_float2(dpA.y, dpA.y);
            const uint32_t hA = __float_as_uint(dpA.z);
            float2 sA[NBL];
#pragma unroll
            for (int k = 0; k < NBL; ++k) sA[k] = make_float2(0.0f, 0.0f);
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                const float2 eA = residual_pair<HALF>(tb[i], PA, v2[i], nDA, hA);
                sA[i / BL] = __ffma2_rn(eA, eA, sA[i / BL]);
            }
#pragma unroll
            for (int k = 0; k < NBL; ++k) {
                keep_smaller(cbest[k], cslot[k], __float_as_uint(sA[k].x), m);
                keep_smaller(cbest[NBL + k], cslot[NBL + k], __float_as_uint(sA[k].y), m);
            }
        }
    } else {
        // one block per thread: lane .x of the SSE pair is member m, lane .y member m + 1 (the
        // slot behind an odd range holds a real member or the copy of the last one: harmless)
        for (int m = 0; m < cnt; m += 2) {
            const float4 dpA = cand[m], dpB = cand[m + 1];
            const float2 PA = make_float2(dpA.y, dpA.y), PB = make_float2(dpB.y, dpB.y);
            const uint32_t nD16 = (__float_as_uint(dpA.z) & 0xFFFFu) | (__float_as_uint(dpB.z) << 16);
            float2 s = make_float2(0.0f, 0.0f);
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                const float2 tA = __fmul2_rn(tb[i], PA), tB = __fmul2_rn(tb[i], PB);   // elements 2i, 2i + 1
                const float2 e0 = residual_two_candidates<HALF>(tA.x, tB.x, v2[i].x, dpA.x, dpB.x, nD16);
                s = __ffma2_rn(e0, e0, s);
                const float2 e1 = residual_two_candidates<HALF>(tA.y, tB.y, v2[i].y, dpA.x, dpB.x, nD16);
                s = __ffma2_rn(e1, e1, s);
            }
            keep_smaller(cbest[0], cslot[0], __float_as_uint(s.x), m);
            keep_smaller(cbest[0], cslot[0], __float_as_uint(s.y), m + 1);
        }
    }
#pragma unroll
    for (int k = 0; k < NBT; ++k)
        if (cbest[k] != 0xFFFFFFFFu) merge_class_winner(best[k], cbest[k], T.member[base + cslot[k]]);
}

// PRUNE: the sweep leaves out, per warp, the candidates that provably cannot change an output
// (see "Pruned sweep" above).
//
// Resident CTAs per SM asked of the register allocator: two (at most 128 registers) for every block
// size up to 32 -- the kernels sit within a few registers of that limit, and falling to one
// resident CTA costs far more (measured: 8 % at B = 16) than the allocator's squeeze; B = 64 needs
// about 170 registers and runs one CTA per SM.
// Elements a thread of k_brute owns: one block for B >= 32, else 32; 16 for B = 2, whose 16
// running minima per 32 elements otherwise leave room for one CTA per SM only (measured: 496 -> 452 us;
// B = 4 and B = 8 lose with 16).
__host__ __device__ constexpr int brute_group_elems(int B) { return B >= 32 ? B : (B == 2 ? 16 : 32); }

constexpr int brute_min_ctas(int B, bool prune) { (void)prune; return B <= 32 ? 2 : 1; }

// The pruned sweep sorts the blocks of a CTA's 256 groups by magnitude when a thread holds several blocks.
__host__ __device__ constexpr bool brute_sorted(int B, bool prune) { return prune && B < 32; }

// Dynamic shared memory of the sorted mode.  The tile holds the CTA's 256 groups as binary32, one padded row
// per group (so that both a thread's own row and rows gathered at random spread over the banks); once
// every thread has taken its blocks the same memory receives the results (code bytes, scale bytes, block
// SSEs, each at the block's original position).  Bins and permutation have memory of their own.
template <int B>
struct BruteTile {
    static constexpr int G = brute_group_elems(B);
    static constexpr int NBT = G / B;                       // blocks per thread (only used for B < 32)
    static constexpr int ROW = G + 1;
    static constexpr int BINS = 1024;                       // exponent and two significand bits of the block maximum
    static constexpr size_t TILE_BYTES = (size_t)kThreads * ROW * 4;
    static constexpr size_t OUT_SCALES = (size_t)kThreads * G / 2;            // after the code bytes
    static constexpr size_t OUT_SSE = OUT_SCALES + (size_t)kThreads * NBT;    // a multiple of 256
    static constexpr size_t OUT_BYTES = OUT_SSE + (size_t)kThreads * NBT * 4;
    static constexpr size_t HIST_OFF = (TILE_BYTES + 15) / 16 * 16;
    static constexpr size_t PERM_OFF = HIST_OFF + (size_t)BINS * 4;
    static constexpr size_t BYTES = PERM_OFF + (size_t)kThreads * NBT * 2;
    static_assert(OUT_BYTES <= TILE_BYTES, "the results fit into the tile's memory");
    static_assert(kThreads * NBT <= 65536 && BINS == 4 * kThreads, "16-bit block indices; four bins per thread");
};

template <int DT, int B, int FMT, bool PRUNE>
__global__ void __launch_bounds__(kThreads, brute_min_ctas(B, PRUNE)) k_brute(QuantArgs p) {
    constexpr bool ONEBLK = (B >= 32);        // the thread owns exactly one block
    constexpr int G = brute_group_elems(B);     // elements per thread
    constexpr int NP = G / 2;                 // pairs per thread
    constexpr int BL = ONEBLK ? NP : B;         // elements of one block inside one half
    constexpr int NBL = NP / BL;              // blocks per half (1 when ONEBLK)
    constexpr int NBT = ONEBLK ? 1 : 2 * NBL;   // blocks per thread
    constexpr int NCLS = (FMT == kUE8M0) ? 1 : 8;
    constexpr float kTiny = 2.168404344971009e-19f;  // 2^-62

    __shared__ BruteTables T;
    wait_for_prior_grid();
    release_dependents();
    const float g = p.d_global_scale ? *p.d_global_scale : p.global_scale;
    const int first = (p.prevent_zero && FMT != kUE8M0) ? 1 : 0;
    build_brute_tables<FMT, PRUNE>(T, g, first);


    // With PRUNE the loop is uniform per warp (lanes past the end repeat the warp's first group
    // and store nothing), so that the warp can agree on the candidates it leaves out.
    //
    // SORTED (PRUNE with several blocks per thread, B <= 16): what a warp may leave out is decided by the
    // smallest and the largest block maximum it holds, and with a handful of small blocks per lane a warp
    // of unsorted blocks holds nearly the whole range of the tensor.  So the CTA first sorts the blocks of
    // its 256 groups by magnitude (a counting sort on the exponent and two significand bits of the block
    // maximum, in shared memory), every thread takes NBT neighbours of the sorted order, and the results
    // travel back through shared memory to the thread that owns the group they belong to, which stores them
    // and adds their SSEs in the original order.  Which thread evaluates a block changes nothing in its
    // result, so the outputs do not depend on the (unordered) ranks inside a bin.  The loop is uniform per
    // CTA in this mode (every barrier below is reached by all 256 threads the same number of times);
    // groups past the end are filled with zeros and store nothing.
    constexpr bool SORTED = brute_sorted(B, PRUNE);
    using Tile = BruteTile<B>;
    extern __shared__ uint4 brute_dyn[];
    [[maybe_unused]] unsigned char* const dyn = reinterpret_cast<unsigned char*>(brute_dyn);
    [[maybe_unused]] float* const tile = reinterpret_cast<float*>(dyn);
    [[maybe_unused]] uint32_t* const hist = reinterpret_cast<uint32_t*>(dyn + Tile::HIST_OFF);
    [[maybe_unused]] uint16_t* const perm = reinterpret_cast<uint16_t*>(dyn + Tile::PERM_OFF);
    __shared__ uint32_t warp_total[kThreads / 32];
    const size_t stride = (size_t)gridDim.x * kThreads;
    const int lane = (PRUNE && !SORTED) ? (threadIdx.x & 31) : 0;
    double sse_sum = 0.0;                  // binary64 sum of the SSEs of this thread's blocks, in the order it stored them
    for (size_t wbase = (size_t)blockIdx.x * kThreads + (SORTED ? 0 : threadIdx.x - lane); wbase < p.n_items; wbase += stride) {
        const bool active = wbase + (SORTED ? threadIdx.x : lane) < p.n_items;
        const size_t grp = SORTED ? wbase + threadIdx.x : (active ? wbase + lane : wbase);
        float2 v2[NP];
        float amax = 0.0f;
        [[maybe_unused]] float amin = 0.0f;   // PRUNE: smallest block maximum of the thread
        bool tiny = false;   // a nonzero magnitude below 2^-62: its quotient by Dref may be inexact
        {
            float v[G];
            if constexpr (SORTED) {
                // own group -> own (padded) row of the tile; bins cleared
                if (active) {
                    load_elems<DT, G>(p.x, grp * G, v);
                } else {
#pragma unroll
                    for (int i = 0; i < G; ++i) v[i] = 0.0f;
                }
#pragma unroll
                for (int i = 0; i < G; ++i) tile[threadIdx.x * Tile::ROW + i] = v[i];
                reinterpret_cast<uint4*>(hist)[threadIdx.x] = make_uint4(0u, 0u, 0u, 0u);
                __syncthreads();
                uint32_t key[NBT], rank[NBT];
#pragma unroll
                for (int kb = 0; kb < NBT; ++kb) {
                    float a = 0.0f;
#pragma unroll
                    for (int i = 0; i < B; ++i) a = fmaxf(a, fabsf(v[kb * B + i]));
                    key[kb] = min(__float_as_uint(a) >> 21, (uint32_t)Tile::BINS - 1u);
                    rank[kb] = atomicAdd(&hist[key[kb]], 1u);
                }
                __syncthreads();
                {   // exclusive prefix sums over the bins: four bins per thread, a scan over the warps' totals
                    const uint4 h = reinterpret_cast<const uint4*>(hist)[threadIdx.x];
                    const uint32_t mine = h.x + h.y + h.z + h.w;
                    uint32_t incl = mine;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                        if ((threadIdx.x & 31) >= o) incl += up;
                    }
                    if ((threadIdx.x & 31) == 31) warp_total[threadIdx.x >> 5] = incl;
                    __syncthreads();
                    uint32_t before = incl - mine;
                    for (int w = 0; w < (int)(threadIdx.x >> 5); ++w) before += warp_total[w];
                    reinterpret_cast<uint4*>(hist)[threadIdx.x] = make_uint4(before, before + h.x, before + h.x + h.y, before + h.x + h.y + h.z);
                }
                __syncthreads();
#pragma unroll
                for (int kb = 0; kb < NBT; ++kb) perm[hist[key[kb]] + rank[kb]] = (uint16_t)(threadIdx.x * NBT + kb);
                __syncthreads();
#pragma unroll
                for (int kb = 0; kb < NBT; ++kb) {
                    const int ob = perm[threadIdx.x * NBT + kb];
                    const float* src = tile + (ob / NBT) * Tile::ROW + (ob % NBT) * B;
#pragma unroll
                    for (int i = 0; i < B; ++i) v[kb * B + i] = src[i];
                }
                __syncthreads();   // the tile has been read: its memory takes the results below
            } else {
                load_elems<DT, G>(p.x, grp * G, v);
            }
            if constexpr (PRUNE && !ONEBLK) {
                float2 bmax[NBL];
#pragma unroll
                for (int k = 0; k < NBL; ++k) bmax[k] = make_float2(0.0f, 0.0f);
#pragma unroll
                for (int i = 0; i < NP; ++i) {
                    v2[i] = make_float2(v[i], v[NP + i]);
                    const float a0 = fabsf(v[i]), a1 = fabsf(v[NP + i]);
                    bmax[i / BL].x = fmaxf(bmax[i / BL].x, a0);
                    bmax[i / BL].y = fmaxf(bmax[i / BL].y, a1);
                    tiny |= (a0 < kTiny && a0 != 0.0f) || (a1 < kTiny && a1 != 0.0f);
                }
                amin = fminf(bmax[0].x, bmax[0].y);
                amax = fmaxf(bmax[0].x, bmax[0].y);
#pragma unroll
                for (int k = 1; k < NBL; ++k) {
                    amin = fminf(amin, fminf(bmax[k].x, bmax[k].y));
                    amax = fmaxf(amax, fmaxf(bmax[k].x, bmax[k].y));
                }
            } else {
#pragma unroll
                for (int i = 0; i < NP; ++i) {
                    // one block per thread: adjacent elements; else element i of either half
                    const float x0 = ONEBLK ? v[2 * i] : v[i], x1 = ONEBLK ? v[2 * i + 1] : v[NP + i];
                    v2[i] = make_float2(x0, x1);
                    const float a0 = fabsf(x0), a1 = fabsf(x1);
                    amax = fmaxf(amax, fmaxf(a0, a1));
                    tiny |= (a0 < kTiny && a0 != 0.0f) || (a1 < kTiny && a1 != 0.0f);
                }
                amin = amax;
            }
        }
        const bool fast_ok = (amax <= kFastMax) && !tiny;

        // best[k]: k < NBL -> block k of the low half, else block k - NBL of the high half
        unsigned long long best[NBT];
#pragma unroll
        for (int k = 0; k < NBT; ++k) best[k] = sse_key(__uint_as_float(0xFFFFFFFFu), first);

        auto class_quotients = [&](int cls, float2 (&tb)[NP]) {
            const float Dr = T.clsD[cls], Rr = T.clsR[cls];
            const float2 nDr2 = make_float2(-Dr, -Dr), Rr2 = make_float2(Rr, Rr);
#pragma unroll
            for (int i = 0; i < NP; ++i)
                tb[i] = quotient_pair(v2[i], nDr2, Rr2);
        };

        if constexpr (!PRUNE) {
            if (fast_ok) {
                for (int cls = 0; cls < NCLS; ++cls) {
                    const int n0 = T.cnt[2 * cls], n1 = T.cnt[2 * cls + 1];
                    if (n0 + n1 == 0) continue;
                    float2 tb[NP];
                    class_quotients(cls, tb);
                    search_list<B, FMT, false>(T, 2 * cls, 0, n0, v2, tb, best);
                    search_list<B, FMT, true>(T, 2 * cls + 1, 0, n1, v2, tb, best);
                }
                // Dref = 1: the elements are their own quotients
                search_list<B, FMT, false>(T, kFlatList, 0, T.cnt[kFlatList], v2, v2, best);
            }
        } else {
            // Warp-wide steps are taken by every lane; lanes on the general path contribute neutral
            // values and evaluate nothing here.
            constexpr uint32_t kFull = 0xFFFFFFFFu, kInfBits = 0x7F800000u;
            const float wmax = __uint_as_float(__reduce_max_sync(kFull, fast_ok ? __float_as_uint(amax) : 0u));
            const uint32_t zero_limit = __float_as_uint(__fmul_rn(4.0f, wmax));   // exact: wmax <= 2^60
            int skipped_min = 256;     // smallest code left out under the zero rule
            uint32_t high_limit = zero_limit, low_limit = 0u;

            // Ranges of one class: [lo, hi) of either kind, and the zero rule's bookkeeping.
            auto class_ranges = [&](int cls, int (&lo)[2], int (&hi)[2]) {
                const uint32_t mant = __float_as_uint(T.clsD[cls]) & 0x007FFFFFu;
                const uint32_t cut_zero = exponent_cut(mant, zero_limit), cut_high = exponent_cut(mant, high_limit);
                const uint32_t cut_low = exponent_cut(mant, low_limit);
#pragma unroll
                for (int kind = 0; kind < 2; ++kind) {
                    const int list = 2 * cls + kind;
                    const int nz = T.below[list][cut_zero];
                    skipped_min = min(skipped_min, nz < T.cnt[list] ? (int)T.member[members_base<FMT>(list) + nz] : 256);
                    hi[kind] = min(nz, (int)T.below[list][cut_high]);
                    lo[kind] = min(hi[kind], (int)T.below[list][cut_low]);
                }
            };

            // First the members of class 0 within nine binades below the zero rule's limit: the
            // optimum of nearly every block lies there, which makes the bounds below tight.
            int lo0[2] = {0, 0}, hi0[2] = {0, 0}, probe[2] = {0, 0};
            const bool have0 = T.cnt[0] + T.cnt[1] > 0;
            if (have0) {
                class_ranges(0, lo0, hi0);
                const uint32_t mant = __float_as_uint(T.clsD[0]) & 0x007FFFFFu;
                const uint32_t cut_probe = exponent_cut(mant, limit_shifted_down(zero_limit, 9));
                probe[0] = min(hi0[0], (int)T.below[0][cut_probe]);
                probe[1] = min(hi0[1], (int)T.below[1][cut_probe]);
                if (fast_ok) {
                    float2 tb[NP];
                    class_quotients(0, tb);
                    search_list<B, FMT, false>(T, 0, probe[0], hi0[0] - probe[0], v2, tb, best);
                    search_list<B, FMT, true>(T, 1, probe[1], hi0[1] - probe[1], v2, tb, best);
                }
            }

            // Bounds from what has been found so far.
            {
                uint32_t ubits = 0u;       // largest best SSE of the thread's blocks
#pragma unroll
                for (int k = 0; k < NBT; ++k) ubits = max(ubits, (uint32_t)(best[k] >> 32));
                float low = __uint_as_float(kInfBits);
                int jt = 4;
                if (fast_ok) {
                    // low rule: a trial D' a little below (a - sqrt(U)) / 6, kept only if it passes the test itself
                    low = 0.0f;
                    if (ubits < kInfBits) {
                        const float r = __fmul_rn(__fsqrt_ru(__uint_as_float(ubits)), 1.0009765625f);
                        const float d = __fmul_rn(__fsub_rn(amin, r), 0.1665f);
                        if (d > 0.0f) {
                            const float e = __fmaf_rn(-6.0f, d, amin);
                            if (e >= 0.0f && __float_as_uint(__fmul_rn(e, e)) > ubits) low = d;
                        }
                    }
                    // high rule: the largest j in {2, 3, 4} whose bound exceeds the best SSE of every block
                    // (a j that fails makes the larger ones fail as well); j = 3 is tried first
                    auto bound_exceeds_best = [&](int j) {
                        const float theta = __fmul_rn(wmax, 1.0f / (float)(1 << j));
                        bool pass = true;
                        if constexpr (!ONEBLK) {
                            float2 z[NBL];
#pragma unroll
                            for (int k = 0; k < NBL; ++k) z[k] = make_float2(0.0f, 0.0f);
#pragma unroll
                            for (int i = 0; i < NP; ++i) {
                                const float2 m = make_float2(fabsf(v2[i].x) <= theta ? v2[i].x : 0.0f,
                                                             fabsf(v2[i].y) <= theta ? v2[i].y : 0.0f);
                                z[i / BL] = __ffma2_rn(m, m, z[i / BL]);
                            }
#pragma unroll
                            for (int k = 0; k < NBL; ++k) {
                                pass &= __float_as_uint(z[k].x) > (uint32_t)(best[k] >> 32);
                                pass &= __float_as_uint(z[k].y) > (uint32_t)(best[NBL + k] >> 32);
                            }
                        } else {
                            float z = 0.0f;
#pragma unroll
                            for (int i = 0; i < NP; ++i) {
                                const float m0 = fabsf(v2[i].x) <= theta ? v2[i].x : 0.0f;
                                z = __fmaf_rn(m0, m0, z);
                                const float m1 = fabsf(v2[i].y) <= theta ? v2[i].y : 0.0f;
                                z = __fmaf_rn(m1, m1, z);
                            }
                            pass = __float_as_uint(z) > (uint32_t)(best[0] >> 32);
                        }
                        return pass;
                    };
                    if (bound_exceeds_best(3))
                        jt = bound_exceeds_best(4) ? 4 : 3;
                    else
                        jt = bound_exceeds_best(2) ? 2 : 0;
                }
                low_limit = __reduce_min_sync(kFull, __float_as_uint(low));
                const int jw = (int)__reduce_min_sync(kFull, (unsigned)jt);
                high_limit = limit_shifted_down(zero_limit, jw);
                if (high_limit == 0u) high_limit = zero_limit;
            }

            // the members of class 0 below the first range that the low rule keeps
            if (have0) {
                const uint32_t cut_low = exponent_cut(__float_as_uint(T.clsD[0]) & 0x007FFFFFu, low_limit);
#pragma unroll
                for (int kind = 0; kind < 2; ++kind) lo0[kind] = min(probe[kind], (int)T.below[kind][cut_low]);
                if (fast_ok && probe[0] - lo0[0] + probe[1] - lo0[1] > 0) {
                    float2 tb[NP];
                    class_quotients(0, tb);    // formed again rather than kept: fewer live registers
                    search_list<B, FMT, false>(T, 0, lo0[0], probe[0] - lo0[0], v2, tb, best);
                    search_list<B, FMT, true>(T, 1, lo0[1], probe[1] - lo0[1], v2, tb, best);
                }
            }
            for (int cls = 1; cls < NCLS; ++cls) {
                if (T.cnt[2 * cls] + T.cnt[2 * cls + 1] == 0) continue;
                int lo[2], hi[2];
                class_ranges(cls, lo, hi);
                if (hi[0] - lo[0] + hi[1] - lo[1] == 0 || !fast_ok) continue;
                float2 tb[NP];
                class_quotients(cls, tb);
                search_list<B, FMT, false>(T, 2 * cls, lo[0], hi[0] - lo[0], v2, tb, best);
                search_list<B, FMT, true>(T, 2 * cls + 1, lo[1], hi[1] - lo[1], v2, tb, best);
            }
            // Flat list.  Its members with a subnormal D lie below every normal low limit; the ones
            // with the multiplier 0 fall under the zero rule.
            if (low_limit >= 0x00800000u) {
                skipped_min = min(skipped_min, T.flat_zero_min);
            } else if (fast_ok) {
                search_list<B, FMT, false>(T, kFlatList, 0, T.cnt[kFlatList], v2, v2, best);
            }
            if (fast_ok && skipped_min < 256) {
                // all-zero quantization: e = v, summed in element order like every other candidate
                if constexpr (!ONEBLK) {
                    float2 s0[NBL];
#pragma unroll
                    for (int k = 0; k < NBL; ++k) s0[k] = make_float2(0.0f, 0.0f);
#pragma unroll
                    for (int i = 0; i < NP; ++i) s0[i / BL] = __ffma2_rn(v2[i], v2[i], s0[i / BL]);
#pragma unroll
                    for (int k = 0; k < NBL; ++k) {
                        const unsigned long long k0 = sse_key(s0[k].x, skipped_min), k1 = sse_key(s0[k].y, skipped_min);
                        if (k0 < best[k]) best[k] = k0;
                        if (k1 < best[NBL + k]) best[NBL + k] = k1;
                    }
                } else {
                    float s0 = 0.0f;
#pragma unroll
                    for (int i = 0; i < NP; ++i) {
                        s0 = __fmaf_rn(v2[i].x, v2[i].x, s0);
                        s0 = __fmaf_rn(v2[i].y, v2[i].y, s0);
                    }
                    const unsigned long long k0 = sse_key(s0, skipped_min);
                    if (k0 < best[0]) best[0] = k0;
                }
            }
        }

        // general path (IEEE division), candidate by candidate: threads that hold a magnitude above
        // 2^60 or a nonzero one below 2^-62
        const int n_general = fast_ok ? 0 : num_codes(FMT);
        for (int c = first; c < n_general; ++c) {
            const float D = T.D[c];
            if (!(fabsf(D) <= 3.402823466e38f)) continue;  // decode scale overflowed: not usable
            if constexpr (!ONEBLK) {
#pragma unroll
                for (int k = 0; k < NBL; ++k) {
                    const unsigned long long k0 = sse_key(general_sse<B, NP>(v2, k * BL, 0, D), c);
                    const unsigned long long k1 = sse_key(general_sse<B, NP>(v2, k * BL, 1, D), c);
                    if (k0 < best[k]) best[k] = k0;
                    if (k1 < best[NBL + k]) best[NBL + k] = k1;
                }
            } else {
                float s = 0.0f;
#pragma unroll
                for (int i = 0; i < NP; ++i) {
                    const float a = v2[i].x, b = v2[i].y;
                    const float2 q = round_e2m1x2(quotient_general(a, D), quotient_general(b, D));
                    const float e0 = __fmaf_rn(-q.x, D, a);
                    s = __fmaf_rn(e0, e0, s);
                    const float e1 = __fmaf_rn(-q.y, D, b);
                    s = __fmaf_rn(e1, e1, s);
                }
                const unsigned long long k0 = sse_key(s, c);
                if (k0 < best[0]) best[0] = k0;
            }
        }

        // final encode with the winners
        uint32_t packed[G / 8];
        uint32_t sc[(NBT + 3) / 4];
        uint32_t sw[NBT];
#pragma unroll
        for (int k = 0; k < (NBT + 3) / 4; ++k) sc[k] = 0;
        if constexpr (ONEBLK) {
            const int code = (int)(best[0] & 0xFFu);
            const float D = T.D[code];
            const float R = T.R[code];
            const bool fast = (R != 0.0f) && (amax <= kFastMax);
            sc[0] = (uint32_t)code;
            sw[0] = (uint32_t)(best[0] >> 32);
#pragma unroll
            for (int k = 0; k < G / 8; ++k) {
                float t[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 a = v2[4 * k + i];
                    t[2 * i] = fast ? quotient_corrected(a.x, D, R) : quotient_general(a.x, D);
                    t[2 * i + 1] = fast ? quotient_corrected(a.y, D, R) : quotient_general(a.y, D);
                }
                packed[k] = pack_e2m1x8(t[0], t[1], t[2], t[3], t[4], t[5], t[6], t[7]);
            }
        } else {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float t[NP];
#pragma unroll
                for (int k = 0; k < NBL; ++k) {
                    const int kb = h * NBL + k;   // block index inside the thread
                    const int code = (int)(best[kb] & 0xFFu);
                    const float D = T.D[code];
                    const float R = T.R[code];
                    const bool fast = (R != 0.0f) && (amax <= kFastMax);
#pragma unroll
                    for (int i = 0; i < BL; ++i) {
                        const float a = h ? v2[k * BL + i].y : v2[k * BL + i].x;
                        t[k * BL + i] = fast ? quotient_corrected(a, D, R) : quotient_general(a, D);
                    }
                    sc[kb / 4] |= (uint32_t)code << (8 * (kb % 4));
                    sw[kb] = (uint32_t)(best[kb] >> 32);
                }
#pragma unroll
                for (int k = 0; k < NP / 8; ++k)
                    packed[h * (NP / 8) + k] = pack_e2m1x8(t[8 * k], t[8 * k + 1], t[8 * k + 2], t[8 * k + 3], t[8 * k + 4],
                                                           t[8 * k + 5], t[8 * k + 6], t[8 * k + 7]);
            }
        }
        if constexpr (SORTED) {
            // results to the blocks' original positions, then every thread fetches those of its own group
            unsigned char* const oc = dyn;
            unsigned char* const os = dyn + Tile::OUT_SCALES;
            uint32_t* const oe = reinterpret_cast<uint32_t*>(dyn + Tile::OUT_SSE);
#pragma unroll
            for (int kb = 0; kb < NBT; ++kb) {
                const int ob = perm[threadIdx.x * NBT + kb];
                if constexpr (B == 2) oc[ob] = (unsigned char)(packed[kb / 4] >> (8 * (kb % 4)));
                else if constexpr (B == 4) reinterpret_cast<uint16_t*>(oc)[ob] = (uint16_t)(packed[kb / 2] >> (16 * (kb % 2)));
                else if constexpr (B == 8) reinterpret_cast<uint32_t*>(oc)[ob] = packed[kb];
                else reinterpret_cast<uint2*>(oc)[ob] = make_uint2(packed[2 * kb], packed[2 * kb + 1]);
                os[ob] = (unsigned char)(sc[kb / 4] >> (8 * (kb % 4)));
                oe[ob] = sw[kb];
            }
            __syncthreads();
#pragma unroll
            for (int k = 0; k < G / 8; ++k) packed[k] = reinterpret_cast<const uint32_t*>(oc)[threadIdx.x * (G / 8) + k];
#pragma unroll
            for (int k = 0; k < (NBT + 3) / 4; ++k) sc[k] = 0;
#pragma unroll
            for (int kb = 0; kb < NBT; ++kb) {
                sc[kb / 4] |= (uint32_t)os[threadIdx.x * NBT + kb] << (8 * (kb % 4));
                sw[kb] = oe[threadIdx.x * NBT + kb];
            }
            __syncthreads();   // before the next trip writes the tile
        }
        if (!PRUNE || active) {
            store_bytes<G / 2>(p.codes + grp * (G / 2), packed);
            store_bytes<NBT>(p.scales + grp * NBT, sc);
            if (p.block_sse) store_bytes<4 * NBT>(p.block_sse + grp * NBT, sw);
#pragma unroll
            for (int k = 0; k < NBT; ++k) sse_sum = __dadd_rn(sse_sum, (double)__uint_as_float(sw[k]));
        }
    }
    if (p.mse_partials != nullptr) {   // launch-uniform: fused tensor-MSE partial sum of this CTA
        __syncthreads();               // the tables are no longer read: their memory serves as scratch
        const double total = cta_sum_fixed_order(sse_sum, reinterpret_cast<double*>(&T));
        if (threadIdx.x == 0) p.mse_partials[p.mse_first + blockIdx.x] = total;
    }
}

// ------------------------------------------------------------------------------------------------
// The blocks past the last whole per-thread group (block sizes up to 16 only): one block per
// thread, general path.
// ------------------------------------------------------------------------------------------------
template <int DT, int B, int FMT>
__global__ void k_brute_tail(QuantArgs p) {
    const size_t b = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    float my_sse = 0.0f;
    if (b < p.n_items) {
    const size_t blk = p.first_item + b;
    const float g = p.d_global_scale ? *p.d_global_scale : p.global_scale;
    const int first = (p.prevent_zero && FMT != kUE8M0) ? 1 : 0;
    float v[B];
    load_elems<DT, B>(p.x, blk * B, v);
    unsigned long long best = sse_key(__uint_as_float(0xFFFFFFFFu), first);
    for (int c = first; c < num_codes(FMT); ++c) {
        const float D = __fmul_rn(scale_value(FMT, c), g);
        if (!(fabsf(D) <= 3.402823466e38f)) continue;
        float s = 0.0f;
#pragma unroll
        for (int i = 0; i < B; i += 2) {
            const float2 q = round_e2m1x2(quotient_general(v[i], D), quotient_general(v[i + 1], D));
            const float e0 = __fmaf_rn(-q.x, D, v[i]);
            s = __fmaf_rn(e0, e0, s);
            const float e1 = __fmaf_rn(-q.y, D, v[i + 1]);
            s = __fmaf_rn(e1, e1, s);
        }
        const unsigned long long k = sse_key(s, c);
        if (k < best) best = k;
    }
    const int code = (int)(best & 0xFFu);
    const float D = __fmul_rn(scale_value(FMT, code), g);
    uint32_t packed[(B + 7) / 8];
#pragma unroll
    for (int k = 0; k < (B + 7) / 8; ++k) packed[k] = 0;
#pragma unroll
    for (int k = 0; k < B / 2; ++k)
        packed[k / 4] |= pack_e2m1x2(quotient_general(v[2 * k], D), quotient_general(v[2 * k + 1], D)) << (8 * (k % 4));
    store_bytes<B / 2>(p.codes + blk * (B / 2), packed);
    p.scales[blk] = (uint8_t)code;
    if (p.block_sse) p.block_sse[blk] = __uint_as_float((uint32_t)(best >> 32));
    my_sse = __uint_as_float((uint32_t)(best >> 32));
    }
    // fused tensor-MSE partial sum: the kernel is one warp, every lane takes part (idle lanes add 0)
    if (p.mse_partials != nullptr) warp_sum_to_partial(p, my_sse);
}

template <int DT, int B, int FMT, bool PRUNE>
static cudaError_t launch_brute_inst(const QuantArgs& a, cudaStream_t stream) {
    static std::atomic<int> ctas_per_sm[kMaxDevices];   // first-use cache; racing threads store the same value
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    constexpr size_t kDynBytes = brute_sorted(B, PRUNE) ? BruteTile<B>::BYTES : 0;   // the sorted mode's tile, bins, permutation
    int resident = ctas_per_sm[dev].load(std::memory_order_relaxed);
    if (resident == 0) {
        if (kDynBytes > 0) {
            err = cudaFuncSetAttribute(k_brute<DT, B, FMT, PRUNE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDynBytes);
            if (err != cudaSuccess) return err;
        }
        int n = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k_brute<DT, B, FMT, PRUNE>, kThreads, kDynBytes);
        if (err != cudaSuccess) return err;
        resident = n > 0 ? n : 1;
        ctas_per_sm[dev].store(resident, std::memory_order_relaxed);
    }
    constexpr size_t G = brute_group_elems(B);    // elements per thread of k_brute
    const size_t n_blocks = a.n_items;
    const size_t n_groups = n_blocks * B / G;
    const size_t done = n_groups * G / B;
    // The blocks past the last whole group go to the one-warp tail kernel.  With fused MSE partial sums it
    // runs first and owns partial 0; the CTAs of the main kernel own the partials from 1 on.
    auto launch_tail = [&]() -> cudaError_t {
        if constexpr (B < 32) {
            if (done < n_blocks) {
                QuantArgs t = a;
                t.first_item = done;
                t.n_items = n_blocks - done;
                t.mse_first = 0;
                k_brute_tail<DT, B, FMT><<<1, 32, 0, stream>>>(t);
                count_launch();
                return cudaGetLastError();
            }
        }
        return cudaSuccess;
    };
    if (a.mse_partials) {
        err = launch_tail();
        if (err != cudaSuccess) return err;
    }
    if (n_groups > 0) {
        QuantArgs m = a;
        m.n_items = n_groups;
        m.mse_first = (done < n_blocks) ? 1 : 0;
        const size_t want = (n_groups + kThreads - 1) / kThreads;
        size_t cap = (size_t)sm_count(dev) * (size_t)resident;
        if (a.mse_partials && cap > (size_t)kMsePartials - 1) cap = kMsePartials - 1;
        const unsigned grid = (unsigned)(want < cap ? want : cap);
        err = launch_pdl(k_brute<DT, B, FMT, PRUNE>, grid, kThreads, kDynBytes, stream, m);
        count_launch();
        if (err != cudaSuccess) return err;
        if (a.mse_n_partials) *a.mse_n_partials = (int)grid + m.mse_first;
    } else if (a.mse_n_partials) {
        *a.mse_n_partials = (done < n_blocks) ? 1 : 0;
    }
    if (!a.mse_partials) err = launch_tail();
    return err;
}

template <int DT, int B, bool PRUNE>
static cudaError_t launch_brute_fmt(const QuantArgs& a, int fmt, cudaStream_t s) {
    switch (fmt) {
    case kUE8M0: return launch_brute_inst<DT, B, kUE8M0, PRUNE>(a, s);
    case kUE4M3: return launch_brute_inst<DT, B, kUE4M3, PRUNE>(a, s);
    default: return launch_brute_inst<DT, B, kUE5M3, PRUNE>(a, s);
    }
}

template <int DT, bool PRUNE>
static cudaError_t launch_brute_dt(const QuantArgs& a, int B, int fmt, cudaStream_t s) {
    switch (B) {
    case 2: return launch_brute_fmt<DT, 2, PRUNE>(a, fmt, s);
    case 4: return launch_brute_fmt<DT, 4, PRUNE>(a, fmt, s);
    case 8: return launch_brute_fmt<DT, 8, PRUNE>(a, fmt, s);
    case 16: return launch_brute_fmt<DT, 16, PRUNE>(a, fmt, s);
    case 32: return launch_brute_fmt<DT, 32, PRUNE>(a, fmt, s);
    default: return launch_brute_fmt<DT, 64, PRUNE>(a, fmt, s);
    }
}

}  // namespace mxq
