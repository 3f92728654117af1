// Self-test of the tcgen05 building blocks (tc_common.cuh) on one 128x128x128 problem:
//   D = A * B^T            both operands from TMA-staged, 128-byte-swizzled shared memory
//   E = bf16(D/64) * C^T   A operand from tensor memory (two bf16 per column), B from shared
// The host compares D and E with a plain matrix product.  This pins the descriptor encodings,
// the TMEM layouts and the barrier protocol independently of the attention kernel.
#pragma once
#include "tc_common.cuh"

namespace adaspark {

struct SelftestSmem {
    __nv_bfloat16 a[2][128][64];   // [d panel][row][64 k] : 16 KB per panel
    __nv_bfloat16 b[2][128][64];
    __nv_bfloat16 c[2][128][64];
    uint64_t full, mma1_done, p_ready, mma2_done;
    uint32_t tmem_base;
    int abort_flag;
};

__global__ void __launch_bounds__(128) umma_selftest_kernel(const __grid_constant__ CUtensorMap tmA,
                                                            const __grid_constant__ CUtensorMap tmB,
                                                            const __grid_constant__ CUtensorMap tmC,
                                                            float* __restrict__ d_out, float* __restrict__ e_out,
                                                            int32_t* __restrict__ status) {
    extern __shared__ unsigned char selftest_raw[];
    SelftestSmem& sm = *reinterpret_cast<SelftestSmem*>((reinterpret_cast<uintptr_t>(selftest_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr uint32_t kIdesc = tc::make_idesc_bf16(128, 128);

    if (tid == 0) {
        tc::mbar_init(&sm.full, 1);
        tc::mbar_init(&sm.mma1_done, 1);
        tc::mbar_init(&sm.p_ready, 128);
        tc::mbar_init(&sm.mma2_done, 1);
        sm.abort_flag = 0;
        tc::fence_barrier_init();
    }
    if (warp == 0) tc::tmem_alloc<512>(&sm.tmem_base);
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tbase = sm.tmem_base;
    volatile int* abort_flag = &sm.abort_flag;
    bool ok = true;

    if (tid == 0) {
        tc::mbar_arrive_expect_tx(&sm.full, 6 * 128 * 64 * 2);
        for (int p = 0; p < 2; ++p) {
            tc::tma_load_2d(&sm.a[p][0][0], &tmA, p * 64, 0, &sm.full);
            tc::tma_load_2d(&sm.b[p][0][0], &tmB, p * 64, 0, &sm.full);
            tc::tma_load_2d(&sm.c[p][0][0], &tmC, p * 64, 0, &sm.full);
        }
        ok = tc::mbar_wait(&sm.full, 0, abort_flag);
        if (ok) {
            tc::tc_fence_after_sync();
            for (int ks = 0; ks < 8; ++ks) {
                uint64_t da = tc::make_smem_desc_sw128(smem_u32(&sm.a[ks >> 2][0][0]) + (ks & 3) * 32);
                uint64_t db = tc::make_smem_desc_sw128(smem_u32(&sm.b[ks >> 2][0][0]) + (ks & 3) * 32);
                tc::umma_ss(tbase, da, db, kIdesc, ks > 0);
            }
            tc::umma_commit(&sm.mma1_done);
        }
    }
    __syncwarp();
    ok = tc::mbar_wait(&sm.mma1_done, 0, abort_flag);
    if (ok) {
        tc::tc_fence_after_sync();
        const int row = warp * 32 + lane;
        const uint32_t lane_addr = tbase + ((uint32_t)(warp * 32) << 16);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tc::tmem_ld_32x32(lane_addr + c * 32, r);
            tc::tmem_wait_ld();
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 32; ++i) d_out[row * 128 + c * 32 + i] = __uint_as_float(r[i]);
#pragma unroll
            for (int i = 0; i < 16; ++i)
                pk[i] = pack_bf16x2(__uint_as_float(r[2 * i]) * (1.f / 64.f), __uint_as_float(r[2 * i + 1]) * (1.f / 64.f));
            tc::tmem_st_32x16(lane_addr + 128 + c * 16, pk);
        }
        tc::tmem_wait_st();
        tc::tc_fence_before_sync();
        tc::mbar_arrive(&sm.p_ready);
    }
    if (tid == 0 && ok) {
        ok = tc::mbar_wait(&sm.p_ready, 0, abort_flag);
        if (ok) {
            tc::tc_fence_after_sync();
            for (int ks = 0; ks < 8; ++ks) {
                uint64_t dc = tc::make_smem_desc_sw128(smem_u32(&sm.c[ks >> 2][0][0]) + (ks & 3) * 32);
                tc::umma_ts(tbase + 256, tbase + 128 + ks * 8, dc, kIdesc, ks > 0);
            }
            tc::umma_commit(&sm.mma2_done);
        }
    }
    __syncwarp();
    if (ok) ok = tc::mbar_wait(&sm.mma2_done, 0, abort_flag);
    if (ok) {
        tc::tc_fence_after_sync();
        const int row = warp * 32 + lane;
        const uint32_t lane_addr = tbase + ((uint32_t)(warp * 32) << 16) + 256;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tc::tmem_ld_32x32(lane_addr + c * 32, r);
            tc::tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) e_out[row * 128 + c * 32 + i] = __uint_as_float(r[i]);
        }
    }
    if (!ok && lane == 0) atomicExch(status, 6);
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_dealloc<512>(tbase);
}

// Self-test of the int8 tensor path: D = A * B^T for int8 A, B [128,128] (row-major, 128 bytes per
// row, TMA-staged with the 128-byte swizzle), int32 result.  Pins the kind::i8 instruction descriptor
// and the signedness of the operands.
struct ImmaSelftestSmem {
    unsigned char a[128][128];
    unsigned char b[128][128];
    uint64_t full, mma_done;
    uint32_t tmem_base;
    int abort_flag;
};

__global__ void __launch_bounds__(128) imma_selftest_kernel(const __grid_constant__ CUtensorMap tmA,
                                                            const __grid_constant__ CUtensorMap tmB,
                                                            int32_t* __restrict__ d_out, int32_t* __restrict__ status) {
    extern __shared__ unsigned char imma_raw[];
    ImmaSelftestSmem& sm = *reinterpret_cast<ImmaSelftestSmem*>((reinterpret_cast<uintptr_t>(imma_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr uint32_t kIdesc = tc::make_idesc_s8(128, 128);
    if (tid == 0) {
        tc::mbar_init(&sm.full, 1);
        tc::mbar_init(&sm.mma_done, 1);
        sm.abort_flag = 0;
        tc::fence_barrier_init();
    }
    if (warp == 0) tc::tmem_alloc<128>(&sm.tmem_base);
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tbase = sm.tmem_base;
    volatile int* abort_flag = &sm.abort_flag;
    bool ok = true;
    if (tid == 0) {
        tc::mbar_arrive_expect_tx(&sm.full, 2 * 128 * 128);
        tc::tma_load_2d(&sm.a[0][0], &tmA, 0, 0, &sm.full);
        tc::tma_load_2d(&sm.b[0][0], &tmB, 0, 0, &sm.full);
        ok = tc::mbar_wait(&sm.full, 0, abort_flag);
        if (ok) {
            tc::tc_fence_after_sync();
            for (int ks = 0; ks < 4; ++ks) {   // 32 bytes of k per step
                uint64_t da = tc::make_smem_desc_sw128(smem_u32(&sm.a[0][0]) + ks * 32);
                uint64_t db = tc::make_smem_desc_sw128(smem_u32(&sm.b[0][0]) + ks * 32);
                tc::umma_ss_i8(tbase, da, db, kIdesc, ks > 0);
            }
            tc::umma_commit(&sm.mma_done);
        }
    }
    __syncwarp();
    ok = tc::mbar_wait(&sm.mma_done, 0, abort_flag);
    if (ok) {
        tc::tc_fence_after_sync();
        const int row = warp * 32 + lane;
        const uint32_t lane_addr = tbase + ((uint32_t)(warp * 32) << 16);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tc::tmem_ld_32x32(lane_addr + c * 32, r);
            tc::tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) d_out[row * 128 + c * 32 + i] = (int32_t)r[i];
        }
    }
    if (!ok && lane == 0) atomicExch(status, 6);
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_dealloc<128>(tbase);
}

// One CTA waits, with the kernels' bounded mbarrier wait, on a barrier at which nothing ever arrives.
// The wait gives up after limit_ns, the abort flag makes the second thread leave its wait too, and
// the kernel reports ADASPARK_ERR_TIMEOUT (6) through `status` and returns normally: the same
// give-up path the attention and scoring kernels take when a protocol error starves a wait.
__global__ void wait_timeout_selftest_kernel(unsigned long long limit_ns, int32_t* status, unsigned long long* waited_ns) {
    __shared__ uint64_t never;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        tc::mbar_init(&never, 1);
        abort_flag = 0;
        tc::fence_barrier_init();
    }
    __syncthreads();
    const uint64_t t0 = tc::global_timer_ns();
    // thread 0 owns the limit; thread 32 waits far longer and must be released by the abort flag
    const bool ok = tc::mbar_wait(&never, 0, &abort_flag, threadIdx.x == 0 ? limit_ns : 1000ull * limit_ns);
    const uint64_t t1 = tc::global_timer_ns();
    if (!ok && threadIdx.x == 0) {
        atomicExch(status, 6);
        *waited_ns = t1 - t0;
    }
    if (!ok && threadIdx.x == 32) atomicAdd(status + 1, 1);
}

}  // namespace adaspark
