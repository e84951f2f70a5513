// Context only -- NOT part of libmpq.so and never a backend of the library.
//
// What the bit-plane method costs on this chip is measured against the product of the DECODED
// integers on the 5th-generation tensor cores (Eq. 16-18: the layer's result is an ordinary integer
// dot product of the odd levels q, or of the level indices u with the correction terms of Eq. 17).
// This file is that comparison kernel, written for sm_100a: C[m][n] = sum_t A[m][t] * B[n][t] with
// 8-bit operands and int32 accumulation,
//   - signed form (codes of up to 7 bits): A, B hold q directly (|q| <= 127);
//   - unsigned form (8-bit codes, |q| <= 255 does not fit int8): A, B hold the level indices u in
//     0..255 and the store applies Eq. 17 expanded over the sum,
//         sum q_a q_b = 4 sum u_a u_b - 2 L_b sum u_a - 2 L_a sum u_b + k L_a L_b,
//     with the row sums of u supplied by row_sums_u8 below.
//
// Structure: persistent, one CTA of 192 threads per multiprocessor, each walking 128 x 256 output
// tiles (tile = blockIdx.x + i * gridDim.x).  Warp 0 (one lane) streams 128-byte wide k-blocks of
// both operands through a 4-stage shared-memory ring with TMA (tiled 2-D loads, 128-byte swizzle,
// no multicast; the tensor maps cover this GPU's own memory); warp 1 (one lane) issues tcgen05.mma
// kind::i8 (M = 128, N = 256, K = 32 per instruction, four per k-block) into one of two 256-column
// TMEM accumulators and releases ring slots with tcgen05.commit; warps 2-5 read the finished
// accumulator back with tcgen05.ld (a warp owns the TMEM lanes of its quarter = 32 output rows)
// and store 128-byte row pieces while the next tile is already being multiplied into the other
// accumulator.  Every wait on an mbarrier is bounded: after kSpinLimit polls the CTA raises
// *error_flag, stops issuing work, waits (bounded again) for its copies in flight, frees its TMEM
// and returns.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr int BM = 128, BN = 256, BK = 128;        // BK in bytes = elements
constexpr int STAGES = 4;
constexpr int STAGE_BYTES = (BM + BN) * BK;          // 48 KiB
constexpr int ACCS = 2;                               // accumulators in TMEM: one is stored while the other is filled
constexpr int TMEM_COLS = ACCS * BN;                  // one 32-bit column per output column and accumulator (all 512)
constexpr int kThreads = 192;                         // warp 0 loads, warp 1 issues the tensor-core work, warps 2-5 store
constexpr uint32_t kSpinLimit = 1u << 20;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
// Bounded wait for the phase with the given parity; false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_addr(bar);
    for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_addr(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_addr(bar)) : "memory");
}
// Shared-memory matrix descriptor of a K-major operand tile stored as rows of 128 bytes with the
// 128-byte swizzle (the layout the TMA load above writes): start address / 16, leading offset 1
// (unused for swizzled K-major), stride between 8-row groups 1024 bytes / 16, descriptor version 1
// (sm_100), layout type 2 = 128-byte swizzle.
__device__ __forceinline__ uint64_t umma_desc_k_major_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFF);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor of kind::i8: int32 accumulator, both operands signed or both unsigned
// 8-bit, both K-major, N = BN, M = BM.
__host__ __device__ constexpr uint32_t umma_idesc_i8(bool is_signed) {
    return (2u << 4) | ((is_signed ? 1u : 0u) << 7) | ((is_signed ? 1u : 0u) << 10) | ((uint32_t)(BN >> 3) << 17) |
           ((uint32_t)(BM >> 4) << 24);
}
__device__ __forceinline__ void umma_i8(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
                 ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
                 : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(bar)) : "memory");
}

struct GemmArgs {
    int32_t* c;
    int64_t n;               // row stride of c
    int k_blocks;
    int is_unsigned;
    const int32_t* sums_a;   // unsigned form: sum_t u_a[r][t]
    const int32_t* sums_b;   // ... sum_t u_b[c][t]
    int La, Lb;
    int64_t k;
    int tiles, n_tiles;      // output tiles in all and along n
    int* error_flag;
};

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
i8_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const GemmArgs g) {
    extern __shared__ __align__(1024) unsigned char ring_raw[];
    __shared__ __align__(8) uint64_t full_bar[STAGES], empty_bar[STAGES], acc_full[ACCS], acc_empty[ACCS];
    __shared__ uint32_t tmem_holder;
    __shared__ int failed;

    // 1024-byte aligned ring (the swizzle pattern repeats every 1024 bytes)
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(ring_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    auto has_failed = [&]() { return *(volatile int*)&failed != 0; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int a = 0; a < ACCS; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 4); }   // four epilogue warps
        failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&tmem_holder)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_holder;

    // my tiles: t = blockIdx.x, blockIdx.x + gridDim.x, ...; tile i of mine uses accumulator i & 1
    const int my_tiles = (g.tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    auto tile_origin = [&](int i, int& m0, int& n0) {
        const int t = (int)blockIdx.x + i * (int)gridDim.x;
        n0 = (t % g.n_tiles) * BN;
        m0 = (t / g.n_tiles) * BM;
    };

    if (warp == 0 && lane == 0) {
        // ---- producer: TMA loads of both operands' k-blocks into the ring, tile after tile
        int issued = 0;                                        // k-blocks issued so far, over all my tiles
        for (int i = 0; i < my_tiles && !has_failed(); ++i) {
            int m0, n0;
            tile_origin(i, m0, n0);
            for (int kb = 0; kb < g.k_blocks; ++kb, ++issued) {
                const int s = issued % STAGES;
                if (issued >= STAGES && !mbar_wait(&empty_bar[s], ((issued / STAGES) - 1) & 1)) { atomicExch(&failed, 1); break; }
                if (has_failed()) break;
                unsigned char* a_dst = ring + (size_t)s * STAGE_BYTES;
                mbar_expect_tx(&full_bar[s], STAGE_BYTES);
                tma_load_2d(a_dst, &map_a, kb * BK, m0, &full_bar[s]);
                tma_load_2d(a_dst + BM * BK, &map_b, kb * BK, n0, &full_bar[s]);
            }
        }
        // on failure: wait (bounded) for the copies already issued before the CTA may leave
        if (has_failed()) {
            for (int q = (issued > STAGES ? issued - STAGES : 0); q < issued; ++q) mbar_wait(&full_bar[q % STAGES], (q / STAGES) & 1);
        }
    } else if (warp == 1 && lane == 0) {
        // ---- tensor-core issue: four K = 32 instructions per 128-byte k-block
        const uint32_t idesc = umma_idesc_i8(!g.is_unsigned);
        int consumed = 0;
        for (int i = 0; i < my_tiles && !has_failed(); ++i) {
            const int acc = i & 1;
            // the accumulator is free once the store of my tile i - 2 has read it
            if (i >= ACCS && !mbar_wait(&acc_empty[acc], ((i >> 1) - 1) & 1)) { atomicExch(&failed, 1); break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BN);
            for (int kb = 0; kb < g.k_blocks; ++kb, ++consumed) {
                const int s = consumed % STAGES;
                if (!mbar_wait(&full_bar[s], (consumed / STAGES) & 1)) { atomicExch(&failed, 1); break; }
                if (has_failed()) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_addr = smem_addr(ring + (size_t)s * STAGE_BYTES);
                const uint64_t da = umma_desc_k_major_sw128(a_addr), db = umma_desc_k_major_sw128(a_addr + BM * BK);
#pragma unroll
                for (int j = 0; j < BK / 32; ++j)      // 32 bytes further along k = 2 sixteen-byte units in the start address
                    umma_i8(tmem_d, da + 2 * j, db + 2 * j, idesc, (kb > 0 || j > 0) ? 1u : 0u);
                umma_commit(&empty_bar[s]);            // the slot is free once these instructions have read it
            }
            umma_commit(&acc_full[acc]);               // all instructions issued so far have completed
        }
    } else if (warp >= 2) {
        // ---- store: TMEM -> registers -> global while the next tile is being multiplied.  A warp may read
        // the TMEM lanes 32 (warp % 4) .. + 31 only: warps 2..5 cover the four quarters = the tile's 128 rows
        const int quarter = warp & 3;
        for (int i = 0; i < my_tiles; ++i) {
            const int acc = i & 1;
            bool ok = mbar_wait(&acc_full[acc], (i >> 1) & 1);
            if (!ok) atomicExch(&failed, 1);
            ok = __all_sync(0xffffffffu, ok && !has_failed());         // the loads below are warp-wide
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            int m0, n0;
            tile_origin(i, m0, n0);
            const int row = m0 + quarter * 32 + lane;
            // Eq. 17 summed over k: 4 sum u_a u_b - 2 L_b sum u_a - 2 L_a sum u_b + k L_a L_b.  The result fits
            // int32 (it is the layer's accumulator), so the terms are combined modulo 2^32.
            const uint32_t row_term = g.is_unsigned ? 2u * (uint32_t)g.Lb * (uint32_t)g.sums_a[row] : 0u;
            const uint32_t constant = g.is_unsigned ? (uint32_t)g.k * (uint32_t)g.La * (uint32_t)g.Lb : 0u;
            const uint32_t col_factor = 2u * (uint32_t)g.La;
#pragma unroll 1
            for (int chunk = 0; chunk < BN / 32; ++chunk) {
                uint32_t v[32];
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + chunk * 32);
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                             "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                             "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                             : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                               "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                               "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                               "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                             : "r"(taddr) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                int32_t* dst = g.c + (int64_t)row * g.n + n0 + chunk * 32;
                const int4* col_sums = g.is_unsigned ? reinterpret_cast<const int4*>(g.sums_b + n0 + chunk * 32) : nullptr;
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    uint32_t o[4] = {v[j], v[j + 1], v[j + 2], v[j + 3]};
                    if (g.is_unsigned) {
                        const int4 sb = __ldg(col_sums + j / 4);
                        o[0] = 4u * o[0] - row_term - col_factor * (uint32_t)sb.x + constant;
                        o[1] = 4u * o[1] - row_term - col_factor * (uint32_t)sb.y + constant;
                        o[2] = 4u * o[2] - row_term - col_factor * (uint32_t)sb.z + constant;
                        o[3] = 4u * o[3] - row_term - col_factor * (uint32_t)sb.w + constant;
                    }
                    *reinterpret_cast<int4*>(dst + j) = make_int4((int)o[0], (int)o[1], (int)o[2], (int)o[3]);
                }
            }
            // this warp's quarter of the accumulator has been read: one of the four arrivals that free it
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[acc]);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && failed) atomicExch(g.error_flag, 1);
}

__global__ void row_sums_u8_kernel(const uint8_t* __restrict__ x, int64_t rows, int64_t k, int32_t* __restrict__ sums) {
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int lane = threadIdx.x & 31;
    int32_t s = 0;
    for (int64_t t = lane; t < k; t += 32) s += x[row * k + t];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) sums[row] = s;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [rows][k] bytes, k contiguous; box = box_rows rows x 128 bytes, 128-byte swizzle.
int make_map(EncodeTiledFn encode, CUtensorMap* map, const void* base, int64_t rows, int64_t k, int box_rows) {
    const cuuint64_t dims[2] = {(cuuint64_t)k, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)k};
    const cuuint32_t box[2] = {BK, (cuuint32_t)box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, elem,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS ? 0 : 1;
}

}  // namespace

// Status: 0 ok, 1 null pointer, 2 bad shape (m, k multiples of 128, n a multiple of 256; k < 2^24), 5 alignment
// (operands, output and sums_b 16-byte aligned), 6 CUDA / driver error.  *error_flag (device int, zeroed by the caller)
// is raised by a CTA whose bounded wait ran out.
extern "C" int mpqctx_i8_gemm(const void* a, const void* b, int64_t m, int64_t n, int64_t k, int32_t* c,
                              int is_unsigned, const int32_t* sums_a, const int32_t* sums_b, int La, int Lb,
                              int* error_flag, void* stream) {
    if (!a || !b || !c || !error_flag || (is_unsigned && (!sums_a || !sums_b))) return 1;
    if (m <= 0 || n <= 0 || k <= 0 || m % BM || n % BN || k % BK || k >= (1 << 24) || (m / BM) * (n / BN) >= (1 << 30)) return 2;
    if ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b) | reinterpret_cast<uintptr_t>(c)) & 15u) return 5;
    if (is_unsigned && (reinterpret_cast<uintptr_t>(sums_b) & 15u)) return 5;
    static EncodeTiledFn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) return 6;
        encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    CUtensorMap map_a, map_b;
    if (make_map(encode, &map_a, a, m, k, BM) || make_map(encode, &map_b, b, n, k, BN)) return 6;
    const size_t smem = (size_t)STAGES * STAGE_BYTES + 1024;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(i8_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return 6;
        configured = true;
    }
    GemmArgs g;
    g.c = c; g.n = n; g.k_blocks = (int)(k / BK); g.is_unsigned = is_unsigned; g.sums_a = sums_a; g.sums_b = sums_b;
    g.La = La; g.Lb = Lb; g.k = k; g.error_flag = error_flag;
    g.n_tiles = (int)(n / BN); g.tiles = (int)((m / BM) * (n / BN));
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 6;
    const int ctas = g.tiles < sms ? g.tiles : sms;           // persistent: one CTA per multiprocessor
    i8_gemm_kernel<<<ctas, kThreads, smem, (cudaStream_t)stream>>>(map_a, map_b, g);
    return cudaGetLastError() == cudaSuccess ? 0 : 6;
}

extern "C" int mpqctx_row_sums_u8(const void* x, int64_t rows, int64_t k, int32_t* sums, void* stream) {
    if (!x || !sums) return 1;
    if (rows <= 0 || k <= 0) return 2;
    row_sums_u8_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, (cudaStream_t)stream>>>(static_cast<const uint8_t*>(x), rows, k, sums);
    return cudaGetLastError() == cudaSuccess ? 0 : 6;
}
