// TENSOR family: the wavefront substitution for many channels on the tcgen05
// tensor cores.
//
// With u the unknown, A_delta = L^-1 W_delta the kernel transformed to the
// paper's unit-diagonal form (Section 3) and A_0 = L^-1,
//     u[p] = A_0 rhs[p] - sum_{delta != 0} A_delta u[p - delta]            (Eq. 1 solved for x_q)
// is evaluated anti-diagonal by anti-diagonal (Section 3.3), but in SCATTER form:
// as soon as diagonal d is solved, its contribution to every later diagonal
// d+1 .. d+2(k-1) is added to accumulators that live in tensor memory, one slot
// of C columns per pending diagonal (a ring of S = 2(k-1) slots).  The 128
// accumulator lanes are (image row h, image i of the group): a tap (dh, dw)
// moves a pixel from lane (h, i) to lane (h + dh, i) -- a row offset of the
// shared-memory operand, applied through the start address of its matrix
// descriptor -- and to diagonal d + dh + dw, i.e. to another slot.  One MMA
// therefore serves all taps of one dh whose target slots are adjacent:
//     D[128 lanes x (n slots * C)] += X_d[128 x ci] * (-A_{dh, dw..dw+n-1})[ci x n*C].
// rhs enters the same way through A_0 (which also opens the slot: accumulate = 0).
//
// Precision: products are formed as  hi(w) hi(x)  [tf32 MMA]  +  lo(w) bf(x) + bf(w) lo(x)  [one bf16 MMA
// whose 16-deep contraction holds both correction terms], hi = round to tf32, lo = the bf16 of the remainder,
// bf = the bf16 of the value; the neglected terms are below 2^-18 of a product.  Accumulation is fp32.
//
// The contraction (input channels) is split over the CTAs of a cluster, CS = 8 * NCH channels each: a CTA
// keeps its channels' slice of the transformed kernel in shared memory for the whole launch, computes partial
// sums for ALL output channels, and the partial sums are exchanged once per diagonal through distributed
// shared memory (each CTA finishes its own CS output channels, which are its input channels of the next
// steps).  Only the two taps that reach the next diagonal, (0,1) and (1,0), are issued before that exchange
// is signalled; the others run on the tensor pipe while the exchange is in flight.
//
// Every wait is bounded; when one gives up the CTA raises INVCONV_TIMEOUT and from then on no wait blocks:
// control flow never diverges from the normal path, so all barriers are still served and the kernel ends.
#pragma once

#include <cuda_bf16.h>

#include "common.cuh"
#include "tma.cuh"
#include "umma.cuh"
#include "tensor_plan.h"

namespace invconv {

struct TensorParams {
    const float* rhs;            // y (forward) or grad_x (backward), [B][C][H][W]
    float* out;                  // x or grad_y
    const unsigned char* wop;    // packed kernel: [R][wbytes]
    int B, C, H, W, K;
    int R, I, HP, S, ngroups, ncl, rot;
    unsigned tmem_cols, wbytes, off_stage, off_x, off_y, off_recv, off_bar, stage_img;
};

// ---------------------------------------------------------------------------
// The transformed kernel A[tap][ci][co] (tap = dh*K + dw; tap 0 = L^-1) arrives from team_solve_kernel in the
// tensor-core operand layout, one contiguous block per CTA rank r (input channels 8r .. 8r+7 for NCH = 1):
//   [dh][chunk][kind][plane][row = dw*C + co][16 bytes]
// kind 0 (tf32): plane p holds hi(v) for ci = 4p .. 4p+3;  kind 1 (bf16): plane 0 holds lo(v), plane 1 bf(v)
// for the chunk's 8 input channels.  v = A for tap 0 and -A for every other tap.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b)
{
    const __nv_bfloat162 t = __floats2bfloat162_rn(a, b);      // .x = a (low half), .y = b
    return *reinterpret_cast<const uint32_t*>(&t);
}

// ---------------------------------------------------------------------------
namespace tensor_detail {


constexpr long long kWaitLimit = 1ll << 24;      // SM cycles (about 8 ms) before a wait gives up

// Waits for the phase of `bar` with the given parity; returns at once when the CTA has already given up.
__device__ __forceinline__ void wait_bar(unsigned long long* bar, unsigned parity, volatile int* gave_up)
{
    if (mbar_try_wait(bar, parity)) return;
    if (*gave_up) return;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*gave_up) return;
        if (clock64() - t0 > kWaitLimit) {
            *gave_up = 1;
            raise_status(INVCONV_TIMEOUT);
            return;
        }
    }
}

// One 128-lane row of an A operand: 8 channel values -> tf32 planes, bf16 value plane, bf16 remainder plane.
// `chunk_base` is the shared-memory address of the chunk's block [kind][plane][rows][16 B].
__device__ __forceinline__ void store_operand_row(unsigned char* chunk_base, int rows, int row, const float (&v)[8])
{
    if (!INVCONV_CHECKED(row, rows, 101)) return;
    float hi[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) hi[j] = tf32_hi(v[j]);
    *reinterpret_cast<float4*>(chunk_base + ((size_t)0 * rows + row) * 16) = make_float4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<float4*>(chunk_base + ((size_t)1 * rows + row) * 16) = make_float4(hi[4], hi[5], hi[6], hi[7]);
    uint4 bf, lo;
    bf.x = pack_bf16x2(v[0], v[1]); bf.y = pack_bf16x2(v[2], v[3]);
    bf.z = pack_bf16x2(v[4], v[5]); bf.w = pack_bf16x2(v[6], v[7]);
    lo.x = pack_bf16x2(v[0] - hi[0], v[1] - hi[1]); lo.y = pack_bf16x2(v[2] - hi[2], v[3] - hi[3]);
    lo.z = pack_bf16x2(v[4] - hi[4], v[5] - hi[5]); lo.w = pack_bf16x2(v[6] - hi[6], v[7] - hi[7]);
    *reinterpret_cast<uint4*>(chunk_base + ((size_t)2 * rows + row) * 16) = bf;     // pairs with lo(w)
    *reinterpret_cast<uint4*>(chunk_base + ((size_t)3 * rows + row) * 16) = lo;     // pairs with bf(w)
}

}  // namespace tensor_detail

// CG = C / 16, K = kernel side.  NCH = 1 (eight contraction channels per CTA).
template <int CG, int K>
__global__ void __launch_bounds__(kTensorThreads, 1) tensor_wavefront_kernel(const TensorParams p)
{
    using namespace tensor_detail;
    constexpr int C = CG * 16;
    constexpr int CS = 8;
    constexpr int S = 2 * (K - 1);
    constexpr int R = C / CS;
    constexpr int KC = K * C;
    constexpr int MAXSLOTS = 256 / C;
    extern __shared__ __align__(128) unsigned char tsmem[];
    unsigned char* const smem = tsmem;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int H = p.H, W = p.W, I = p.I;
    const int D = H + W - 1, HALO = (K - 1) * I, ROWS = HALO + 128;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int cluster_id = blockIdx.x / R;

    unsigned char* s_w = smem;
    float* s_stage = reinterpret_cast<float*>(smem + p.off_stage);
    unsigned char* s_x = smem + p.off_x;            // [2][kind][plane][ROWS][16]
    unsigned char* s_y = smem + p.off_y;            // [2][kind][plane][128][16]
    float* s_recv = reinterpret_cast<float*>(smem + p.off_recv);   // [2][R-1][CS/4][128][4]: lanes contiguous, 16 bytes each
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + p.off_bar);
    unsigned long long* wbar = bars + 0;
    unsigned long long* ybar = bars + 1;            // the group's slice of rhs has arrived in the staging buffer
    unsigned long long* accbar = bars + 2;          // the next diagonal's accumulator is complete
    unsigned long long* xfull = bars + 3;           // [2] solved diagonal written as an operand
    unsigned long long* yfull = bars + 5;           // [2] rhs diagonal written as an operand
    unsigned long long* yfree = bars + 7;           // [2] the MMA that read it is done
    unsigned long long* rbar = bars + 9;            // [2] partial sums of the peers have arrived
    unsigned long long* xdone = bars + 11;          // the group's solved slice is complete in the staging buffer
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 12);
    volatile int* gave_up = reinterpret_cast<volatile int*>(bars + 13);

    const unsigned xbuf_bytes = 4u * ROWS * 16, ybuf_bytes = 4u * 128 * 16;
    constexpr unsigned recv_buf_floats = (unsigned)(R - 1) * 128 * CS;
    // Lanes (h, i) with pixel (h, d - h) inside the image form one contiguous range; only they exchange sums.
    auto recv_bytes = [&](int d) {
        const int hmin = d - W + 1 > 0 ? d - W + 1 : 0, hmax = d < H - 1 ? d : H - 1;
        return (unsigned)((R - 1) * (hmax - hmin + 1) * I * CS * 4);
    };

    if (tid == 0) {
        mbar_init(wbar, 1); mbar_init(ybar, 1); mbar_init(accbar, 1);
        mbar_init(xfull + 0, 256); mbar_init(xfull + 1, 256);
        mbar_init(yfull + 0, 128); mbar_init(yfull + 1, 128);
        mbar_init(yfree + 0, 1); mbar_init(yfree + 1, 1);
        mbar_init(rbar + 0, 1); mbar_init(rbar + 1, 1);
        mbar_init(xdone, 256);
        *gave_up = 0;
        fence_mbar_init();
        mbar_expect_tx(rbar + 0, recv_bytes(0));    // armed before any peer can send
        mbar_expect_tx(rbar + 1, recv_bytes(1 % D));
    }
    // zero both solved-diagonal operand buffers once (their first HALO rows stay zero: lanes shifted in from
    // above the image are the zero padding)
    for (unsigned e = tid; e < 2 * xbuf_bytes / 16; e += kTensorThreads) reinterpret_cast<uint4*>(s_x)[e] = make_uint4(0, 0, 0, 0);
    if (warp == 8) umma::tmem_alloc(tmem_slot, p.tmem_cols);
    fence_proxy_async();
    umma::fence_before_sync();
    __syncthreads();
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");     // peers' barriers exist before anything is sent
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    umma::fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    const size_t img_floats = (size_t)C * H * W;
    const unsigned slice_bytes = (unsigned)(CS * H * W * sizeof(float));

    if (warp < 8) {
        // ------------------------------------------------ accumulators -> solved pixels
        // Two threads per accumulator lane: warpgroup wg = warp / 4 takes the partial sums of the peers
        // wg*CG .. wg*CG+CG-1 (8 columns each) and finishes channels 4wg .. 4wg+3 of this CTA's own eight.
        const int wg = warp >> 2;
        const int m = tid & 127, h = m / I, i = m - h * I;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        // where this lane's partial sums land in each peer, and the peer's arrival barrier (buffer 0)
        uint32_t remote_row[CG], remote_bar[CG];
#pragma unroll
        for (int q = 0; q < CG; ++q) {
            const int pr = wg * CG + q;
            const int slot = (int)rank < pr ? (int)rank : (int)rank - 1;
            remote_row[q] = cluster_map_u32(smem_u32(s_recv + (size_t)slot * 128 * CS + (size_t)m * 4), (uint32_t)pr);
            remote_bar[q] = cluster_map_u32(smem_u32(rbar), (uint32_t)pr);
        }
        const uint32_t own_col = rank * CS + wg * 4;
        unsigned nd = 0;            // diagonals processed so far (all groups): buffer = nd & 1, phase = (nd >> 1) & 1
        unsigned ng = 0;            // groups processed so far
        for (int g = cluster_id; g < p.ngroups; g += p.ncl, ++ng) {
            const int img = g * I + i;
            const bool img_ok = img < p.B;
            wait_bar(ybar, ng & 1, gave_up);
            int slot_d = 0;
            for (int d = 0; d < D; ++d, ++nd) {
                const unsigned b = nd & 1, ph = (nd >> 1) & 1;
                wait_bar(accbar, nd & 1, gave_up);
                umma::fence_after_sync();
                uint32_t acc[CG][8], own[4];
                const uint32_t col = (uint32_t)(slot_d * C);
                (void)INVCONV_CHECKED(col + C - 1, p.tmem_cols, 105);
                slot_d = slot_d + 1 == S ? 0 : slot_d + 1;
#pragma unroll
                for (int q = 0; q < CG; ++q) umma::tmem_ld8(lane_addr + col + (wg * CG + q) * 8, acc[q]);
                umma::tmem_ld4(lane_addr + col + own_col, own);
#pragma unroll
                for (int q = 0; q < CG; ++q) umma::tmem_ld_fence(acc[q]);
                umma::tmem_ld_fence(own);
                umma::fence_before_sync();
                // partial sums of the other CTAs' output channels go to their owners
                const uint32_t boff = b * recv_buf_floats * 4, bbar = b * 8;
                const int w = d - h;
                const bool on_diag = h < H && w >= 0 && w < W;
#pragma unroll
                for (int q = 0; q < CG; ++q) {
                    if (wg * CG + q != (int)rank && on_diag) {
                        st_async_f32x4(remote_row[q] + boff, make_float4(__uint_as_float(acc[q][0]), __uint_as_float(acc[q][1]),
                                                                       __uint_as_float(acc[q][2]), __uint_as_float(acc[q][3])), remote_bar[q] + bbar);
                        st_async_f32x4(remote_row[q] + boff + 128 * 16, make_float4(__uint_as_float(acc[q][4]), __uint_as_float(acc[q][5]),
                                                                                  __uint_as_float(acc[q][6]), __uint_as_float(acc[q][7])), remote_bar[q] + bbar);
                    }
                }
                wait_bar(rbar + b, ph, gave_up);
                if (tid == 0) mbar_expect_tx(rbar + b, recv_bytes((d + 2) % D));   // arm the phase two diagonals ahead
                // own channels 4wg .. 4wg+3: sum over the CTAs in rank order
                const float* recv_b = s_recv + b * recv_buf_floats + wg * 128 * 4 + m * 4;
                float4 pa[R - 1];
#pragma unroll
                for (int sl = 0; sl < R - 1; ++sl)
                    pa[sl] = (on_diag && INVCONV_CHECKED((recv_b - s_recv) + (size_t)sl * 128 * CS + 3, 2 * recv_buf_floats, 102))
                                 ? *reinterpret_cast<const float4*>(recv_b + (size_t)sl * 128 * CS) : make_float4(0.f, 0.f, 0.f, 0.f);
                float v[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int pr = 0; pr < R; ++pr) {
                    if (pr == (int)rank) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) v[j] += __uint_as_float(own[j]);
                    }
                    if (pr < R - 1) {
                        // slot pr holds rank pr if that is below this CTA's rank, else rank pr + 1: adding slot pr
                        // after the own term of rank pr keeps the sum in rank order
                        v[0] += pa[pr].x; v[1] += pa[pr].y; v[2] += pa[pr].z; v[3] += pa[pr].w;
                    }
                }
                const bool valid = img_ok && on_diag;
                if (!valid) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) v[j] = 0.f;
                }
                {   // this warpgroup's half of the operand row: tf32 plane wg, 8 bytes of each bf16 plane
                    unsigned char* xb = s_x + b * xbuf_bytes;
                    const int row = HALO + m;
                    (void)INVCONV_CHECKED(row, ROWS, 101);
                    float hi[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) hi[j] = tf32_hi(v[j]);
                    *reinterpret_cast<float4*>(xb + ((size_t)wg * ROWS + row) * 16) = make_float4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<uint2*>(xb + ((size_t)2 * ROWS + row) * 16 + wg * 8) =
                        make_uint2(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]));
                    *reinterpret_cast<uint2*>(xb + ((size_t)3 * ROWS + row) * 16 + wg * 8) =
                        make_uint2(pack_bf16x2(v[0] - hi[0], v[1] - hi[1]), pack_bf16x2(v[2] - hi[2], v[3] - hi[3]));
                }
                fence_proxy_async();
                mbar_arrive(xfull + b);
                if (valid) {
                    const int hh = p.rot ? H - 1 - h : h, ww = p.rot ? W - 1 - w : w;
                    float* dst = s_stage + (size_t)i * p.stage_img + (size_t)(wg * 4) * H * W + (size_t)hh * W + ww;
                    if (INVCONV_CHECKED((dst - s_stage) + (size_t)3 * H * W, (size_t)I * p.stage_img, 103)) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) dst[(size_t)j * H * W] = v[j];
                    }
                }
            }
            fence_proxy_async();          // the staged slice is stored by bulk copies
            mbar_arrive(xdone);
        }
    } else if (warp == 8) {
        // ------------------------------------------------ MMA issue (one thread)
        if (tid == 256) {
            wait_bar(wbar, 0, gave_up);
            const unsigned xplane = ROWS * 16;
            constexpr unsigned wplane = KC * 16;
            // descriptors of row 0 (no lane shift) of buffer 0 / of tap row 0 of dh = 0; everything else is an offset in 16-byte units
            const uint64_t xd_tf = umma::make_desc(smem_u32(s_x) + HALO * 16, xplane);
            const uint64_t xd_bf = umma::make_desc(smem_u32(s_x) + 2 * xplane + HALO * 16, xplane);
            const uint64_t yd_tf = umma::make_desc(smem_u32(s_y), 128 * 16);
            const uint64_t yd_bf = umma::make_desc(smem_u32(s_y) + 2 * 128 * 16, 128 * 16);
            const uint64_t wd_tf = umma::make_desc(smem_u32(s_w), wplane);
            const uint64_t wd_bf = umma::make_desc(smem_u32(s_w) + 2 * wplane, wplane);
            const uint32_t xbuf16 = xbuf_bytes >> 4, ybuf16 = ybuf_bytes >> 4;
            constexpr uint32_t idesc_tf = umma::make_idesc(umma::kFmtTF32, 0), idesc_bf = umma::make_idesc(umma::kFmtBF16, 0);
            constexpr uint32_t cbits = ((uint32_t)C >> 3) << 17;
            const uint64_t w01_tf = wd_tf + (uint64_t)C, w01_bf = wd_bf + (uint64_t)C;                         // dh = 0, dw = 1
            const uint64_t w10_tf = wd_tf + (uint64_t)(4 * (wplane >> 4)), w10_bf = wd_bf + (uint64_t)(4 * (wplane >> 4));   // dh = 1, dw = 0
            unsigned nd = 0, ny = 0;
            // taps (dh, a .. a+n-1) of the solved diagonal d in buffer b -> the slots of diagonals d+dh+a ...;
            // slot_d = d mod S.  Split where the slot ring wraps and at 256 accumulator columns.
            auto window = [&](unsigned b, int d, int slot_d, int dh, int a, int n) {
                const int t0 = d + dh + a;
                if (t0 + n > D) n = D - t0;
                int s0 = slot_d + dh + a;
                if (s0 >= S) s0 -= S;
                const uint64_t atf = xd_tf + (uint64_t)(b * xbuf16) - (uint64_t)(dh * I);
                const uint64_t abf = xd_bf + (uint64_t)(b * xbuf16) - (uint64_t)(dh * I);
                const uint32_t wrow = (uint32_t)(dh * 4) * (wplane >> 4);
                while (n > 0) {
                    int c = n;
                    if (c > S - s0) c = S - s0;
                    if (c > MAXSLOTS) c = MAXSLOTS;
                    const uint32_t dcol = tmem + (uint32_t)(s0 * C);
                    const uint32_t nbits = ((uint32_t)(c * C) >> 3) << 17;
                    if (!INVCONV_CHECKED((s0 + c) * C - 1, p.tmem_cols, 106) || !INVCONV_CHECKED(HALO - dh * I, ROWS - 127, 107) ||
                        !INVCONV_CHECKED((a + c) * C - 1, KC, 108)) break;
                    umma::mma_tf32(dcol, atf, wd_tf + wrow + (uint32_t)(a * C), idesc_tf | nbits, 1u);
                    umma::mma_bf16(dcol, abf, wd_bf + wrow + (uint32_t)(a * C), idesc_bf | nbits, 1u);
                    a += c; n -= c; s0 += c;
                    if (s0 >= S) s0 -= S;
                }
            };
            // rhs of the next diagonal (operand buffer ny & 1) through A_0 = tap (0,0): opens slot `slot`
            auto rhs_tap = [&](int slot) {
                const unsigned b = ny & 1;
                wait_bar(yfull + b, (ny >> 1) & 1, gave_up);
                umma::fence_after_sync();
                const uint32_t dcol = tmem + (uint32_t)(slot * C);
                constexpr uint32_t nbits = ((uint32_t)C >> 3) << 17;
                umma::mma_tf32(dcol, yd_tf + b * ybuf16, wd_tf, idesc_tf | nbits, 0u);
                umma::mma_bf16(dcol, yd_bf + b * ybuf16, wd_bf, idesc_bf | nbits, 1u);
                umma::commit(yfree + b);
                ++ny;
            };
            for (int g = cluster_id; g < p.ngroups; g += p.ncl) {
                for (int t = 0; t < S && t < D; ++t) rhs_tap(t);
                umma::commit(accbar);
                int slot_d = 0;
                for (int d = 0; d < D; ++d, ++nd) {
                    const unsigned b = nd & 1;
                    wait_bar(xfull + b, (nd >> 1) & 1, gave_up);
                    umma::fence_after_sync();
                    if (d + 1 < D) {       // taps (0,1) and (1,0): the next diagonal waits for these only
                        const uint32_t dcol = tmem + (uint32_t)((slot_d + 1 == S ? 0 : slot_d + 1) * C);
                        const uint64_t xo = b ? (uint64_t)xbuf16 : 0ull;
                        umma::mma_tf32(dcol, xd_tf + xo, w01_tf, idesc_tf | cbits, 1u);
                        umma::mma_bf16(dcol, xd_bf + xo, w01_bf, idesc_bf | cbits, 1u);
                        umma::mma_tf32(dcol, xd_tf + xo - (uint64_t)I, w10_tf, idesc_tf | cbits, 1u);
                        umma::mma_bf16(dcol, xd_bf + xo - (uint64_t)I, w10_bf, idesc_bf | cbits, 1u);
                        umma::commit(accbar);
                    }
                    if (d + S < D) rhs_tap(slot_d);
                    if (K > 2) window(b, d, slot_d, 0, 2, K - 2);
                    window(b, d, slot_d, 1, 1, K - 1);
#pragma unroll
                    for (int dh = 2; dh < K; ++dh) window(b, d, slot_d, dh, 0, K);
                    slot_d = slot_d + 1 == S ? 0 : slot_d + 1;
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ right-hand side: load, operand rows, final store
        const int lt = tid - 288;
        const int m = lt, h = m / I, i = m - h * I;
        unsigned ny = 0, ng = 0;
        if (lt == 0) {
            asm volatile("griddepcontrol.wait;" ::: "memory");       // the kernel transform (previous launch) is complete
            mbar_expect_tx(wbar, p.wbytes);
            const unsigned per = p.wbytes / (unsigned)K;
            for (int dh = 0; dh < K; ++dh) bulk_g2s(s_w + (size_t)dh * per, p.wop + (size_t)rank * p.wbytes + (size_t)dh * per, per, wbar);
        }
        for (int g = cluster_id; g < p.ngroups; g += p.ncl, ++ng) {
            const int nimg = min(I, p.B - g * I);
            if (lt == 0) {
                mbar_expect_tx(ybar, (unsigned)nimg * slice_bytes);
                for (int ii = 0; ii < nimg; ++ii)
                    if (INVCONV_CHECKED((size_t)(g * I + ii) * img_floats + (size_t)(rank + 1) * CS * H * W - 1, (size_t)p.B * img_floats, 109))
                        bulk_g2s(s_stage + (size_t)ii * p.stage_img,
                                 p.rhs + (size_t)(g * I + ii) * img_floats + (size_t)rank * CS * H * W, slice_bytes, ybar);
            }
            wait_bar(ybar, ng & 1, gave_up);
            const bool img_ok = i < nimg;
            for (int t = 0; t < D; ++t, ++ny) {
                const unsigned b = ny & 1;
                if (ny >= 2) wait_bar(yfree + b, ((ny >> 1) - 1) & 1, gave_up);
                const int w = t - h;
                float v[CS];
                if (img_ok && h < H && w >= 0 && w < W) {
                    const int hh = p.rot ? H - 1 - h : h, ww = p.rot ? W - 1 - w : w;
                    const float* src = s_stage + (size_t)i * p.stage_img + (size_t)hh * W + ww;
                    const bool inb = INVCONV_CHECKED((src - s_stage) + (size_t)(CS - 1) * H * W, (size_t)I * p.stage_img, 104);
#pragma unroll
                    for (int j = 0; j < CS; ++j) v[j] = inb ? src[(size_t)j * H * W] : 0.f;
                } else {
#pragma unroll
                    for (int j = 0; j < CS; ++j) v[j] = 0.f;
                }
                store_operand_row(s_y + b * ybuf_bytes, 128, m, v);
                fence_proxy_async();
                mbar_arrive(yfull + b);
            }
            // the solved slice leaves once every diagonal has been written to the staging buffer
            if (lt == 0) {
                wait_bar(xdone, ng & 1, gave_up);
                for (int ii = 0; ii < nimg; ++ii)
                    bulk_s2g(p.out + (size_t)(g * I + ii) * img_floats + (size_t)rank * CS * H * W,
                             s_stage + (size_t)ii * p.stage_img, slice_bytes);
                bulk_commit();
                bulk_wait_read0();
            }
        }
    }
    // no CTA leaves while a peer may still send to it; tensor memory is returned by the warp that took it
    umma::fence_before_sync();
    __syncthreads();
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (warp == 8) {
        umma::fence_after_sync();
        umma::tmem_dealloc(tmem, p.tmem_cols);
    }
}

}  // namespace invconv
