// LUT3 weight-only decode mat-vec (App. C.2 "Kernel specification"), the batch-1 path:
//   Y[b][n] = bf16( s * sum_blk d_blk * sum_{k in blk} G[idx(n,k)] * X[b][k] )
// Weights stream from HBM as three index words per 32 weights + one signed E4M3 scale per 16 weights
// (3.5 bit per weight); they are dequantised in registers and accumulated in fp32 on the plain ALUs.
//
// Work split.  K is cut into slices of 1024 weights; warp w of a row group owns slice w for every row,
// lane l owns the 32 weights of word triplet 32 w + l.  A lane therefore keeps its 32 activations in
// registers (as fp32 pairs) for the whole kernel and reads, per row, one 32-bit word of each of the three
// word regions and two scale bytes, all at fixed offsets inside the 448-byte block of its slice.  Four rows
// of all slices are contiguous in memory and arrive with one bulk copy into a shared-memory ring.  Partial
// sums meet in a warp butterfly, then across the warps of the group through shared memory.
//
// Dequantisation.  The device bit order (lut3_locate) stores indices as nibbles, so one AND per word (three
// shifts and three bitwise ops for the last eight weights) gives selector words whose bytes each hold the
// indices of two neighbouring weights; one byte-permute turns such a byte into the shared-memory address of a
// table of level pairs (the fp16 codebook widened to fp32; entry stride 256 B, one 8-byte slot per lane, so
// lookups never collide on a bank); the pair is multiplied into the accumulator pair with one packed fp32 FMA.
// (Looking up fp16 pairs and widening them in registers halves the shared-memory traffic but costs two more
// instructions per pair: measured 14 weights/clk/SM.)
//
// What bounds it.  One 64-bit shared-memory lookup per weight pair caps this formulation at 32 weights per
// clock per SM; the kernel reaches 16-18 (about 2 TB/s of weight traffic), HBM would deliver 52.  The
// streaming skeleton alone (ring, word reads, reduction, no lookups) runs at 4.1 TB/s.
#include "dq_common.cuh"
#include "dq_tcgen05.cuh"

namespace dq {

namespace {

constexpr int kRowsPerIter = 4;
constexpr int kSmallCta = 512;                         // register budget of 128 per thread
constexpr int kMidCta = 576;
constexpr uint32_t kTableWindowAddr = 65536;          // table base inside the CTA's shared window (64 KiB aligned)
constexpr uint32_t kTableBytes = 65536;               // 256 entries x 256 B
constexpr uint32_t kDynSmemBytes = 231424;           // the whole opt-in shared memory of an SM less 1 KiB
constexpr uint32_t kCtrlBytes = 4096;                // reduction buffers, levels, mbarriers

__device__ __forceinline__ uint32_t lds_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr)
{
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr) : "memory");
    return v;
}
// the table is written once before the first lookup and never changes: plain (non-volatile) loads
__device__ __forceinline__ unsigned long long lds_u64(uint32_t addr)
{
    unsigned long long v;
    asm volatile("ld.shared.u64 %0, [%1];" : "=l"(v) : "r"(addr));
    return v;
}
// packed fp32 pair FMA: acc += a * b on both halves
__device__ __forceinline__ void ffma2(unsigned long long &acc, unsigned long long a, unsigned long long b)
{
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi)
{
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// two signed E4M3 bytes -> two floats
__device__ __forceinline__ void e4m3x2_to_f32(uint32_t two, float &d0, float &d1)
{
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((unsigned short)two));
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.f32.f16 %0, l;\n\tcvt.f32.f16 %1, h;\n\t}"
        : "=f"(d0), "=f"(d1) : "r"(h2));
}

// bounded mbarrier wait with back-off between polls
__device__ __forceinline__ bool gemv_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    if (tc::mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t it = 0;
    while (true) {
        __nanosleep(40);
        if (tc::mbar_try(bar, parity)) return true;
        if ((++it & 63u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > tc::kWaitBudgetCycles) { *abort_flag = 1; return false; }
        }
    }
}

// R rows in lockstep.  All lookups of a 16-weight block (8 pairs per row) are issued before the
// first FMA that consumes them, so that the shared-memory latency is paid once per block and not
// once per pair.  out[r][t] = d0 * sum(block 0) + d1 * sum(block 1) of row r against column t.
template <int BT, int R>
__device__ __forceinline__ void dot32_rows(const uint32_t (&p0)[R], const uint32_t (&p1)[R], const uint32_t (&p2)[R],
                                           const uint32_t (&sc)[R], uint32_t lane_base,
                                           const unsigned long long (&xs)[BT][16], float (&out)[R][BT])
{
    float d[R][2];
    uint32_t sel[R][4];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        lut3_selectors(p0[r], p1[r], p2[r], sel[r]);
        e4m3x2_to_f32(sc[r], d[r][0], d[r][1]);
#pragma unroll
        for (int t = 0; t < BT; ++t) out[r][t] = 0.0f;
    }
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) {          // pairs 0..7 are block 0, pairs 8..15 block 1
        unsigned long long gp[R][8];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int g = 2 * blk + h;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                // selector word g: byte j holds the indices of weight pair 4g + j as nibbles (idx_b << 4 | idx_a)
                const uint32_t u = sel[r][g];
#pragma unroll
                for (int j = 0; j < 4; ++j)      // address = table base | byte j of u << 8 | lane * 8
                    gp[r][4 * h + j] = lds_u64(__byte_perm(u, lane_base, 0x7604 | (j << 4)));
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int t = 0; t < BT; ++t) {
                // two accumulator pairs per row shorten the dependent FMA chain
                unsigned long long acc0 = 0ull, acc1 = 0ull;
#pragma unroll
                for (int q = 0; q < 8; q += 2) {
                    ffma2(acc0, gp[r][q], xs[t][8 * blk + q]);
                    ffma2(acc1, gp[r][q + 1], xs[t][8 * blk + q + 1]);
                }
                float a0, a1, b0, b1;
                unpack_f32x2(acc0, a0, a1);
                unpack_f32x2(acc1, b0, b1);
                out[r][t] = fmaf(d[r][blk], (a0 + a1) + (b0 + b1), out[r][t]);
            }
    }
}

template <int BT, int MAXT>
__global__ void __launch_bounds__(MAXT, 1)
gemv_lut3_kernel(const uint8_t *__restrict__ lut, const uint8_t *__restrict__ table_img,
                 const PackedHeader *__restrict__ hdr,
                 const __nv_bfloat16 *__restrict__ X, int64_t ldx, int b0,
                 int B, __nv_bfloat16 *__restrict__ Y, int64_t ldy, int N, int K, int W, int G, int S,
                 StatusWord *status)
{
    extern __shared__ __align__(16) uint8_t smem_raw[];
    const uint32_t win0 = (uint32_t)__cvta_generic_to_shared(smem_raw);
    // shared window: [win0, +4 KiB) control | ring part A up to 64 KiB | table 64..128 KiB | ring part B
    float *red = reinterpret_cast<float *>(smem_raw);                       // [G][2][rows][BT][W] partial sums
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_raw + 2048 + 64);
    const uint32_t table_bar = win0 + 2048 + 96;                            // arrival of the table image
    const uint32_t bar0 = win0 + 2048 + 128;                                // full[G*S], empty[G*S]

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int grp = warp / W;
    const int w = warp - grp * W;
    const int nw = K / 32;
    const int widx = w * 32 + lane;                          // plane word this lane owns in every row
    const bool active = widx < nw;                           // a partial last slice is zero padded in memory

    const uint32_t lane_base = kTableWindowAddr | (uint32_t)(lane * 8);
    const int group_threads = W * 32;
    const int nblocks = N / kRowsPerIter;                    // N % 16 == 0
    const int stride = gridDim.x * G;
    const uint32_t row_bytes = (uint32_t)W * kLutBlockBytes;
    const uint32_t chunk_bytes = kRowsPerIter * row_bytes;   // one stage of one group: 4 whole rows
    const uint32_t ringA0 = (win0 + kCtrlBytes + 15u) & ~15u;
    const uint32_t nA = (kTableWindowAddr - ringA0) / chunk_bytes;
    const uint32_t ringB0 = kTableWindowAddr + kTableBytes;
    auto chunk_addr = [&](int s) {                            // stage s of this group, as a shared-window address
        const uint32_t idx = (uint32_t)(s * G + grp);
        return idx < nA ? ringA0 + idx * chunk_bytes : ringB0 + (idx - nA) * chunk_bytes;
    };
    auto full_bar = [&](int s) { return bar0 + 8u * (uint32_t)(grp * S + s); };
    auto empty_bar = [&](int s) { return bar0 + 8u * (uint32_t)(G * S + grp * S + s); };

    // the ring as the host sized it must fit this CTA's shared window (uniform decision, before any barrier)
    {
        const uint32_t last = (uint32_t)(S * G - 1);
        const uint32_t end = last < nA ? ringA0 + (last + 1) * chunk_bytes : ringB0 + (last - nA + 1) * chunk_bytes;
        if (end > win0 + kDynSmemBytes || ringA0 + kCtrlBytes > kTableWindowAddr || 2u * G * S * 8u + 2048 + 128 > kCtrlBytes) {
            if (threadIdx.x == 0) { atomicExch(&status->status, (int)DQ_ERR_INTERNAL); atomicExch(&status->detail, 0x31000); }
            return;
        }
    }
    if (threadIdx.x == 0) {
        *abort_flag = 0;
        tc::mbar_init(table_bar, 1);
        for (int i = 0; i < G * S; ++i) {
            tc::mbar_init(bar0 + 8u * i, 1);                       // full: one producer arrival + bytes
            tc::mbar_init(bar0 + 8u * (G * S + i), (uint32_t)W);   // empty: one arrival per consumer warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    // the 64 KiB pair table was built at pack time: one bulk copy brings it in while set-up continues
    if (threadIdx.x == 0) {
        tc::mbar_expect_tx(table_bar, kTableBytes);
        tc::bulk_load(kTableWindowAddr, table_img, kTableBytes, table_bar);
    }

    // producer of this group: lane 0 of its first warp streams whole row blocks into the ring
    const bool producer = (w == 0 && lane == 0);
    const int first = blockIdx.x * G + grp;
    if (producer) {
        for (int s = 0; s < S; ++s) {
            const int rb = first + s * stride;
            if (rb < nblocks) {
                tc::mbar_expect_tx(full_bar(s), chunk_bytes);
                tc::bulk_load(chunk_addr(s), lut + (size_t)rb * chunk_bytes, chunk_bytes, full_bar(s));
            }
        }
    }

    // Programmatic dependent launch: everything above touches only the packed weights, which no kernel
    // running now can be writing (packing ends with a separate trailing launch).  Activations and output
    // may belong to the kernel before this one in the stream, so wait for it here; the kernel after this
    // one may begin its own set-up as soon as every CTA of this grid has got this far.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // this lane's 32 activations per batch column, widened to fp32 pairs, kept in registers
    unsigned long long xs[BT][16];
#pragma unroll
    for (int t = 0; t < BT; ++t) {
        const bool col_ok = active && (b0 + t < B);
        const uint4 *xp = reinterpret_cast<const uint4 *>(X + (int64_t)(col_ok ? b0 + t : 0) * ldx + (int64_t)(active ? widx : 0) * 32);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint4 v = col_ok ? __ldg(xp + q) : make_uint4(0, 0, 0, 0);
            const uint32_t ww[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int z = 0; z < 4; ++z)
                xs[t][4 * q + z] = pack_f32x2(__uint_as_float(ww[z] << 16), __uint_as_float(ww[z] & 0xFFFF0000u));
        }
    }
    const float s_w = hdr->s;
    bool ok = true;
    {   // table image must have landed before the first lookup
        uint32_t good = 1;
        if (lane == 0) good = gemv_wait(table_bar, 0u, abort_flag) ? 1u : 0u;
        ok = __shfl_sync(0xffffffffu, good, 0) != 0;
    }

    int it = 0, stage = 0;
    uint32_t phase = 0;
    const uint32_t lane_off = (uint32_t)w * kLutBlockBytes + (uint32_t)lane * 4;
    const uint32_t sc_off = (uint32_t)w * kLutBlockBytes + kLutScaleOff + (uint32_t)lane * 2;
    for (int rb = first; rb < nblocks; rb += stride, ++it) {
        // a wait that ran out poisons the rest of the run, but every warp keeps walking the same
        // iterations (with zeros) so that nobody is left alone at a named barrier
        // one lane polls (with back-off) so that waiting warps do not flood the shared-memory pipe
        if (ok) {
            uint32_t good = 1;
            if (lane == 0) good = gemv_wait(full_bar(stage), phase, abort_flag) ? 1u : 0u;
            ok = __shfl_sync(0xffffffffu, good, 0) != 0;
        }
        const uint32_t base = chunk_addr(stage);
        uint32_t p0[kRowsPerIter], p1[kRowsPerIter], p2[kRowsPerIter], sc[kRowsPerIter];
#pragma unroll
        for (int r = 0; r < kRowsPerIter; ++r) {
            const uint32_t a = base + (uint32_t)r * row_bytes;
            p0[r] = ok ? lds_u32(a + lane_off) : 0u;
            p1[r] = ok ? lds_u32(a + lane_off + 128) : 0u;
            p2[r] = ok ? lds_u32(a + lane_off + 256) : 0u;
            sc[r] = ok ? lds_u16(a + sc_off) : 0u;
        }
        // the stage is in registers: release it, and let the producer refill it with the block S steps ahead
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(empty_bar(stage));
        if (producer) {
            const int nxt = rb + S * stride;
            if (nxt < nblocks && ok) {
                if (gemv_wait(empty_bar(stage), phase, abort_flag)) {
                    tc::mbar_expect_tx(full_bar(stage), chunk_bytes);
                    tc::bulk_load(base, lut + (size_t)nxt * chunk_bytes, chunk_bytes, full_bar(stage));
                }
            }
        }
        __syncwarp();

        float v[kRowsPerIter][BT];
        {
#pragma unroll
            for (int r2 = 0; r2 < kRowsPerIter; r2 += 2) {
                const uint32_t q0[2] = {p0[r2], p0[r2 + 1]}, q1[2] = {p1[r2], p1[r2 + 1]};
                const uint32_t q2[2] = {p2[r2], p2[r2 + 1]}, qs[2] = {sc[r2], sc[r2 + 1]};
                float o[2][BT];
                dot32_rows<BT, 2>(q0, q1, q2, qs, lane_base, xs, o);
#pragma unroll
                for (int t = 0; t < BT; ++t) { v[r2][t] = o[0][t]; v[r2 + 1][t] = o[1][t]; }
            }
        }
        // butterfly: afterwards lane l holds the warp total of row ((l>>4)&1)*2 + ((l>>3)&1)
#pragma unroll
        for (int t = 0; t < BT; ++t) {
#pragma unroll
            for (int st = 0; st < 2; ++st) {
                const int off = 16 >> st, cnt = 2 >> st;
                const bool upper = (lane & off) != 0;
#pragma unroll
                for (int i = 0; i < cnt; ++i) {
                    const float send = upper ? v[i][t] : v[i + cnt][t];
                    const float keep = upper ? v[i + cnt][t] : v[i][t];
                    v[i][t] = keep + __shfl_xor_sync(0xffffffffu, send, off);
                }
            }
            v[0][t] += __shfl_xor_sync(0xffffffffu, v[0][t], 4);
            v[0][t] += __shfl_xor_sync(0xffffffffu, v[0][t], 2);
            v[0][t] += __shfl_xor_sync(0xffffffffu, v[0][t], 1);
        }
        float *rbuf = red + ((grp * 2 + (it & 1)) * kRowsPerIter * BT) * W;
        if ((lane & 7) == 0) {
            const int row_l = ((lane >> 4) & 1) * 2 + ((lane >> 3) & 1);
#pragma unroll
            for (int t = 0; t < BT; ++t) rbuf[(row_l * BT + t) * W + w] = v[0][t];
        }
        // the warps of this row group meet; groups use separate named barriers
        asm volatile("bar.sync %0, %1;" ::"r"(grp + 1), "r"(group_threads) : "memory");
        if (w == 0 && lane < kRowsPerIter * BT) {
            const int row_l = lane / BT, t = lane % BT;
            float tot = 0.0f;
            for (int ww = 0; ww < W; ++ww) tot += rbuf[(row_l * BT + t) * W + ww];
            const int row = rb * kRowsPerIter + row_l;
            if (b0 + t < B) Y[(int64_t)(b0 + t) * ldy + row] = __float2bfloat16_rn(tot * s_w);
        }
        if (++stage == S) { stage = 0; phase ^= 1u; }
    }
    if (*abort_flag) {
        // a wait ran out: let copies in flight land, then report; other warps of the group may be
        // parked at their named barrier, so leave through the CTA-wide exit only
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        if (lane == 0) atomicExch(&status->status, (int)DQ_ERR_TIMEOUT);
        if (lane == 0) atomicExch(&status->detail, 0x30000 | (int)blockIdx.x);
    }
}

}  // namespace

template <int BT, int MAXT>
static cudaError_t launch_one(const GemvArgs &a, int b0, int grid, int threads, int W, int G, int S,
                              cudaStream_t stream)
{
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(gemv_lut3_kernel<BT, MAXT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kDynSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    // launched so that its set-up (barriers, lookup table, first weight blocks) may overlap the tail of
    // the kernel before it in the stream; the kernel itself waits before it touches X or Y
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = kDynSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_lut3_kernel<BT, MAXT>, a.lut, a.table, a.hdr,
                              reinterpret_cast<const __nv_bfloat16 *>(a.X), (int64_t)a.ldx, b0, (int)a.B,
                              reinterpret_cast<__nv_bfloat16 *>(a.Y), (int64_t)a.ldy, (int)a.N, (int)a.K, W, G, S,
                              a.status);
}

cudaError_t launch_gemv_lut3(const GemvArgs &a, cudaStream_t stream)
{
    const int K = (int)a.K, N = (int)a.N, B = (int)a.B;
    const int W = (K + 1023) / 1024;                  // warps per row group (one 1024-weight slice each)
    if (W > 32) return cudaErrorInvalidValue;
    int G = 16 / W;                                   // row groups per CTA: up to 512 threads
    if (G < 1) G = 1;
    if (G > 15) G = 15;                               // one named barrier per group
    const int threads = G * W * 32;
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int nblocks = N / kRowsPerIter;
    int grid = (nblocks + G - 1) / G;
    if (grid > sms) grid = sms;
    // ring depth: as many 4-row stages per group as fit around the 64 KiB table (at least 2, at most 8)
    const uint32_t chunk = (uint32_t)kRowsPerIter * W * kLutBlockBytes;
    const uint32_t nA = (kTableWindowAddr - 1024 - kCtrlBytes - 16) / chunk;
    const uint32_t nB = (kDynSmemBytes - (kTableWindowAddr + kTableBytes)) / chunk;
    int S = (int)((nA + nB) / (uint32_t)G);
    if (S > 8) S = 8;
    if (S < 2) return cudaErrorInvalidValue;
    for (int b0 = 0; b0 < B; b0 += 2) {
        cudaError_t e;
        if (threads <= kSmallCta) {
            e = (B - b0 >= 2) ? launch_one<2, kSmallCta>(a, b0, grid, threads, W, G, S, stream)
                              : launch_one<1, kSmallCta>(a, b0, grid, threads, W, G, S, stream);
        } else if (threads <= kMidCta) {               // 17 or 18 slices (K up to 18432): 112 registers per thread
            e = (B - b0 >= 2) ? launch_one<2, kMidCta>(a, b0, grid, threads, W, G, S, stream)
                              : launch_one<1, kMidCta>(a, b0, grid, threads, W, G, S, stream);
        } else {
            e = (B - b0 >= 2) ? launch_one<2, 1024>(a, b0, grid, threads, W, G, S, stream)
                              : launch_one<1, 1024>(a, b0, grid, threads, W, G, S, stream);
        }
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace dq
