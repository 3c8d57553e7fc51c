// tcgen05 / TMEM / TMA tensor-core path for sm_100a: implicit-GEMM 3x3 convolution (forward,
// data gradient, weight gradient) and the sharded fully-connected GEMMs, all bf16 x bf16 -> fp32.
//
// One kernel template, three operand arrangements ("modes"):
//   FWD   : D[pixel, n]  = sum_{tap, c} act[pixel + tap, c] * W[n, tap, c]       A K-major,  B K-major
//   DGRAD : D[pixel, n]  = sum_{tap, k} dy[pixel - tap, k]  * W[k, tap, n]       A K-major,  B MN-major
//   WGRAD : D[m, n]      = sum_{pixel} dy[pixel, m] * act[pixel + tap, n]        A MN-major, B MN-major
// A fully-connected layer is the same thing with one tap and 1x1 "images" (pixel = batch row).
//
// Every operand tile is a set of 128-byte rows fetched by TMA (cp.async.bulk.tensor, 4-D boxes,
// SWIZZLE_128B; out-of-bounds coordinates read zeros, which implements the convolution padding,
// ragged tile edges and ragged reduction tails) into a ring of shared-memory stages guarded by
// mbarriers.  One elected lane issues tcgen05.mma (M = 128, N = BN, K = 16 per instruction) into a TMEM
// accumulator; tcgen05.commit releases a stage back to the TMA producer; four epilogue warps read
// the accumulator with tcgen05.ld and apply bias+ReLU / the ReLU mask / the split-sum store.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM allocator + MMA issuer,
// warps 2..5 = epilogue (TMEM lane quadrant = warp_id % 4).
//
// Hang safety: every mbarrier wait is bounded (iteration cap and a wall-clock deadline); a wait
// that gives up records a code in the model's device status word and the CTA drains and exits
// normally (TMEM is always released), so a broken pipeline turns into SB_ERR_TIMEOUT on the
// host instead of a stuck GPU.
//
// Large forward / data-gradient grids with 256-wide N tiles, and the weight gradients of layers with
// 256+ output channels, run on CTA pairs (umma_pair_kernel, tcgen05.mma.cta_group::2): two
// neighbouring M tiles share one fetch of the other operand, half of it per CTA.
// No load uses multicast; the only multicast is the pair kernel's tcgen05.commit, which releases a
// ring slot in both CTAs of the pair.
//
// Epilogues: bf16 output tiles with whole rows are staged in the drained operand ring and leave by
// TMA stores; a forward tile of a layer that a 2x2 max-pool follows is pooled from that stage in the
// same kernel (pool_from_stage); split reductions write float partial tiles that an ordered reduce
// kernel finishes.  The MMA and TMA issue loops run as converged warps with the instruction
// predicated on one elected lane (descriptors in uniform registers).
#include "sb_umma.h"
#include "sb_tcgen05.cuh"

#include <cstdio>
#include <cstdlib>
#include <cstring>

namespace sb {

enum { MODE_FWD = 0, MODE_DGRAD = 1, MODE_WGRAD = 2 };
enum { UEPI_BIAS_ACT = 0, UEPI_MASK = 1, UEPI_F32 = 2 };

struct UmmaParams {
    int mode, ntaps;
    // pixel-box geometry of the activation-side operand(s): box = bw x bh x bn pixels
    int bw, bh, bn;
    int W, H, N;
    int tiles_w, tiles_h, tiles_n;
    // FWD / DGRAD reduction: kchunks 64-wide chunks per tap; w_cols = row length of one tap in the weight matrix
    int kchunks, w_cols;
    // output columns
    int n_total;          // valid output columns (FWD: Cout, DGRAD: Cin, WGRAD: Cin)
    int shards, tiles_per_shard;  // N-tile enumeration per model shard (FWD of a sharded FC layer); shards=1 otherwise
    // WGRAD
    int m_total;          // rows of the weight gradient (Cout / out-features)
    int m_shards, m_tiles_per_shard;
    int tap_group;        // WGRAD: filter taps per CTA: 1, 3 (one filter row; Cin = 64, N tile = 3 x 64 columns) or 2 (Cin = 128,
                          // N tile = 2 x 128 columns; the fifth group holds tap 8 alone)
    int splits, chunks_per_split, total_chunks;   // split of the reduction (k-iterations) over blockIdx.z
    int stages;           // depth of the shared-memory ring (<= MAX_STAGES)
    float* part;          // FWD/DGRAD with splits > 1: raw float partial sums [split][pixel][n_total]
    // epilogue
    int epi, relu, out_f32;
    int tma_out;          // FWD/DGRAD, bf16 output, no split: the tile is staged in shared memory and written by TMA stores (map C)
    int w_first;          // FWD/DGRAD: the first ring of WEIGHT loads is issued before the wait for the predecessor kernel (the host sets it
                          // only when that kernel cannot have written the weights), the activation loads after it
    void* out;            // FWD/DGRAD: [pixels][ldc] bf16 (or float when out_f32); WGRAD: float partial sums
    __nv_bfloat16* pool_out;   // FWD with tma_out, conv layer followed by a 2x2 max-pool: the pool layer's output [N][H/2][W/2][ldc]
    uint8_t* pool_idx;         // ... and its argmax bytes (dh*2+dw), same shape; nullptr = no fused pool
    long ldc;
    const float* bias;
    const __nv_bfloat16* ref;   // UEPI_MASK: same layout as out; nullptr = no mask
    long split_stride;    // WGRAD: floats between split partial buffers
    int bias_fused;       // WGRAD: the centre-tap CTAs of the first N tile also sum dy over the pixels (the bias gradient)
    long bias_off;        // WGRAD: float offset of the bias-gradient vector inside one split buffer
    uint32_t* status;
    int wg_sweep;         // WGRAD: the float tile leaves through shared memory in contiguous row segments (wgrad_sweep_epilogue)
    // WGRAD with the update folded in (sgd_w != nullptr): the sweep applies v <- mu v + g, w <- w - lr v to the parameters at
    // the tile's offsets (same element offsets as in `out`) and refreshes their bf16 copy instead of storing g
    float *sgd_w, *sgd_v;
    __nv_bfloat16* sgd_s;
    float sgd_lr, sgd_mu;
    // Reciprocals for the divisions on the CTAs' start-up and epilogue paths (filled by launch_op from the fields above):
    // q = n / d as __umulhi(n, mul) with mul = 2^32 / d + 1, exact while n * d < 2^32; mul = 0 stands for d = 1.
    uint32_t rcp_tiles_w, rcp_tiles_wh, rcp_bw, rcp_bwbh, rcp_wb, rcp_wbhb;   // (wb, hb = bw / 2, bh / 2: the pooled box)
    // Halo variant of the 3x3 FWD / DGRAD kernel (umma_halo_kernel): the pixel box lies in shared memory as [h][n][w] rows
    // (tile row = wi + bw * (ni + bn * hi)), one activation fetch of bh + 2 image rows serves the three taps of a filter column.
    int hn_order;         // 1: tile rows in (h, n, w) order; 0: (n, h, w)
    int a_stages;         // depth of the activation (halo) ring; `stages` is then the depth of the weight ring
    uint32_t rcp_bwbn;    // reciprocal of bw * bn (hn_order)
    uint32_t rcp_mtiles;  // reciprocal of tiles_w * tiles_h * tiles_n (persistent halo kernel: tile index -> N tile)
#ifdef SB_CTA_TIMING
    unsigned long long* timing;   // development builds only: per-CTA phase timestamps, 16 per CTA, first 1024 CTAs
    int dbg_skip;                 // development builds only (halo kernel, timing experiments, WRONG results): bit 0 = no activation
                                  // loads after the first ring, bit 1 = no weight loads after the first ring
    unsigned long long* trace;    // development builds only: [0] = record counter, records of 4 words from word 8 on (one per CTA)
#endif
};

// Per-CTA phase stamps: compiled in only with -DSB_CTA_TIMING (a development aid; the shipped kernels carry none).
#ifdef SB_CTA_TIMING
#define SB_TLOG(cond, slot, val) do { if (tlog && (cond)) tlog[slot] = (unsigned long long)(val); } while (0)
#define SB_TRACE_BEGIN() const unsigned long long trace_t0 = globaltimer_ns(); unsigned long long trace_a = 0, trace_b = 0, trace_c = 0
#define SB_TRACE_STAMP(var) do { if (p.trace != nullptr && threadIdx.x == 0) var = globaltimer_ns(); } while (0)
#define SB_TRACE_END(kind) do { if (p.trace != nullptr && threadIdx.x == 0) { \
        const unsigned long long ti_ = atomicAdd(p.trace, 1ull); \
        if (ti_ < 40000ull) { unsigned long long* r_ = p.trace + 8 + 6 * ti_; unsigned smid_; asm volatile("mov.u32 %0, %%smid;" : "=r"(smid_)); \
            r_[0] = trace_t0; r_[1] = globaltimer_ns(); \
            r_[2] = (unsigned long long)smid_ | ((unsigned long long)(kind) << 16) | ((unsigned long long)p.mode << 24) | ((unsigned long long)(gridDim.x * gridDim.y * gridDim.z) << 32); \
            r_[3] = (unsigned long long)(unsigned)p.total_chunks | ((unsigned long long)(unsigned)p.n_total << 32); \
            r_[4] = ((trace_a - trace_t0) & 0xffffffffull) | (((trace_b - trace_t0) & 0xffffffffull) << 32); r_[5] = trace_c - trace_t0; } } } while (0)
#else
#define SB_TLOG(cond, slot, val) do { } while (0)
#define SB_TRACE_BEGIN() do { } while (0)
#define SB_TRACE_STAMP(var) do { } while (0)
#define SB_TRACE_END(kind) do { } while (0)
#endif

__host__ __device__ __forceinline__ uint32_t fast_rcp(uint32_t d) { return d <= 1u ? 0u : (uint32_t)(0x100000000ull / d) + 1u; }
__device__ __forceinline__ int fast_div(int n, uint32_t mul) { return mul == 0u ? n : (int)__umulhi((uint32_t)n, mul); }
// the same with one correction step: the estimate is never low and at most one high for any n < 2^31, so this is exact
// for every tile index (fast_div alone is exact while n * d < 2^32: rows of a tile, pooled pixels of a tile)
__device__ __forceinline__ int fast_div_exact(int n, uint32_t mul, int d)
{
    if (mul == 0u) return n;
    uint32_t q = __umulhi((uint32_t)n, mul);
    if (q * (uint32_t)d > (uint32_t)n) --q;
    return (int)q;
}

constexpr int UMMA_THREADS = 192;
constexpr int A_STAGE_BYTES = 16384;   // 128 rows x 128 B (K-major) or 2 boxes of 64 rows x 128 B (MN-major)

constexpr int CTRL_BYTES = 2048;       // [0,512) barriers + flags, [512,1536) bias (FWD)
constexpr int MAX_STAGES = 8;
template <int MODE, int BN> struct Cfg {
    static constexpr int B_STAGE_BYTES = BN * 128;
    static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    static constexpr int MAX_STAGES_FIT = (BN >= 256) ? 4 : (BN >= 192 ? 5 : (BN >= 128 ? 6 : 8));   // what fits in 227 KB
    static constexpr int TMEM_COLS = BN == 192 ? 256 : BN;    // allocations are powers of two
    static constexpr int smem_bytes(int stages) { return stages * STAGE_BYTES + 1024 /*alignment slack*/ + CTRL_BYTES; }
};

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }   // the 128 epilogue threads (warps 2..5)

// Weight-gradient epilogue through shared memory: the float tile leaves in whole, contiguous row segments.
// The accumulator row of a thread is one gradient ROW (ldc floats apart from the next thread's), so storing it
// straight from registers gives every warp instruction 32 separate 16-byte pieces (measured 2.3 TB/s on a 411 MB
// gradient).  Here the tile goes through the drained operand ring in slabs of 64 columns -- thread r writes its 64 floats
// as 16-byte chunks, chunk c at position c ^ (r & 7) of its 8-chunk group, which spreads a warp's stores over all banks
// -- and is then swept row by row: half a warp takes one row's 256 contiguous bytes, so every global access of a warp
// is two whole 256-byte runs.
// With room for two slabs in the drained ring (two_bufs) consecutive slabs alternate between them, and one barrier per slab
// is enough: whoever has passed the barrier of slab j has finished sweeping slab j - 1, whose buffer slab j + 1 reuses.
template <int BN>
__device__ __forceinline__ void wgrad_sweep_epilogue(const UmmaParams& p, uint32_t taddr, uint8_t* stage, int row, int m0, int m_hi,
                                                      int n0, int n_hi, size_t tile_off, int slab_mult = 1, bool two_bufs = false)
{
    const int t128 = threadIdx.x - 64, q = t128 >> 5, lane = t128 & 31;
    const int hl = lane & 15, sub = lane >> 4;
    const uint32_t stage_base = smem_u32(stage);
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += 64) {
        if (n0 + c0 >= n_hi) break;                       // (uniform)
        const uint32_t stage_s = stage_base + ((two_bufs && (c0 & 64)) ? 32768u : 0u);
#pragma unroll
        for (int cc = 0; cc < 64; cc += 32) {
            uint32_t v[2][16];
            tmem_ld16(taddr + c0 + cc, v[0]);             // two loads per wait
            tmem_ld16(taddr + c0 + cc + 16, v[1]);
            tmem_ld_wait();
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t ch = (uint32_t)((cc + 16 * h) / 4 + j);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stage_s + (uint32_t)row * 256u + ((ch ^ (uint32_t)(row & 7)) << 4)),
                                 "r"(v[h][4 * j]), "r"(v[h][4 * j + 1]), "r"(v[h][4 * j + 2]), "r"(v[h][4 * j + 3]) : "memory");
                }
        }
        epi_bar_sync();
        const int col = n0 + c0 + 4 * hl;
        if (col < n_hi) {
#pragma unroll 2
            for (int rr = q * 2 + sub; rr < 128; rr += 8) {
                if (m0 + rr >= m_hi) break;
                float4 g;
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(g.x), "=f"(g.y), "=f"(g.z), "=f"(g.w)
                             : "r"(stage_s + (uint32_t)rr * 256u + (((uint32_t)hl ^ (uint32_t)(rr & 7)) << 4)));
                const size_t off = tile_off + (size_t)rr * p.ldc + (size_t)(c0 * slab_mult) + 4 * hl;   // (slab_mult: 64-column slabs three taps apart)
                *(float4*)((float*)p.out + off) = g;
            }
        }
        if (!two_bufs) epi_bar_sync();                    // the slab may be overwritten
    }
}

// The same sweep with the SGD-momentum update folded in (FC layers in the fused step): instead of storing the gradient
// tile, v <- mu v + g and w <- w - lr v are applied to the parameters at the tile's offsets and their bf16 copy is
// refreshed -- the operations of the stand-alone update kernel in the same order, so the bits are the same, while the
// float gradient is neither written nor read back (8 of 26 bytes per parameter).  The w and v boxes of a 64-column slab
// (128 rows x 256 bytes each, float tensor maps over the master weights and the momentum buffer) are fetched ahead by
// TMA into two slab buffers behind the control block: slabs 0 and 1 are requested before the main loop starts, slab
// j + 2 when slab j has been swept, so a CTA has 64 - 128 KB of parameter loads in flight while it multiplies, drains
// and sweeps.  (One 256-byte bulk copy per row and array, 256 per slab, kept the TMA unit busy for ~5 us per slab.)
constexpr int UPD_SLAB_BYTES = 65536;                 // per slab buffer: w rows [128][256 B], then v rows [128][256 B]
constexpr int UPD_EXTRA_SMEM = 2 * UPD_SLAB_BYTES;
__device__ __forceinline__ void upd_request_slab(const CUtensorMap* mapW, const CUtensorMap* mapV, uint8_t* buf, uint64_t* bar, int col, int m0)
{
    // one thread: a 64-column x 128-row box of w and one of v (rows past the matrix read as zeros and are never stored)
    mbar_expect_tx(bar, (uint32_t)UPD_SLAB_BYTES);
    tma_load_4d(mapW, buf, bar, col, m0, 0, 0);
    tma_load_4d(mapV, buf + 32768, bar, col, m0, 0, 0);
}
template <int BN>
__device__ __forceinline__ bool wgrad_sweep_update_epilogue(const UmmaParams& p, const CUtensorMap* mapW, const CUtensorMap* mapV, uint32_t taddr,
                                                             uint8_t* stage, uint8_t* slab_buf, uint64_t* slab_bar, int row, int m0, int m_hi, int n0,
                                                             int n_hi, size_t tile_off)
{
    const uint32_t slab_s = smem_u32(slab_buf);
    const int t128 = threadIdx.x - 64, q = t128 >> 5, lane = t128 & 31;
    const int hl = lane & 15, sub = lane >> 4;
    const uint32_t stage_s = smem_u32(stage);
    bool ok = true;
#pragma unroll 1
    for (int j = 0; j < BN / 64; ++j) {
        const int c0 = 64 * j;
        if (n0 + c0 >= n_hi) break;                       // (uniform)
        const uint32_t buf_s = slab_s + (uint32_t)(j & 1) * (uint32_t)UPD_SLAB_BYTES;
#pragma unroll
        for (int cc = 0; cc < 64; cc += 16) {
            uint32_t v[16];
            tmem_ld16(taddr + c0 + cc, v);
            tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t ch = (uint32_t)(cc / 4 + k);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stage_s + (uint32_t)row * 256u + ((ch ^ (uint32_t)(row & 7)) << 4)),
                             "r"(v[4 * k]), "r"(v[4 * k + 1]), "r"(v[4 * k + 2]), "r"(v[4 * k + 3]) : "memory");
            }
        }
        // the slab's parameter rows have landed (every thread waits: it reads other threads' rows)
        if (ok) ok = mbar_wait(&slab_bar[j & 1], (uint32_t)((j >> 1) & 1));
        epi_bar_sync();
        if (ok) {
#pragma unroll 4
            for (int rr = q * 2 + sub; rr < 128; rr += 8) {
                if (m0 + rr >= m_hi) break;
                float4 g, w, v;
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(g.x), "=f"(g.y), "=f"(g.z), "=f"(g.w)
                             : "r"(stage_s + (uint32_t)rr * 256u + (((uint32_t)hl ^ (uint32_t)(rr & 7)) << 4)));
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(w.x), "=f"(w.y), "=f"(w.z), "=f"(w.w)
                             : "r"(buf_s + (uint32_t)rr * 256u + ((uint32_t)hl << 4)));
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                             : "r"(buf_s + 32768u + (uint32_t)rr * 256u + ((uint32_t)hl << 4)));
                v.x = fmaf(p.sgd_mu, v.x, g.x); v.y = fmaf(p.sgd_mu, v.y, g.y); v.z = fmaf(p.sgd_mu, v.z, g.z); v.w = fmaf(p.sgd_mu, v.w, g.w);
                w.x = fmaf(-p.sgd_lr, v.x, w.x); w.y = fmaf(-p.sgd_lr, v.y, w.y); w.z = fmaf(-p.sgd_lr, v.z, w.z); w.w = fmaf(-p.sgd_lr, v.w, w.w);
                const size_t off = tile_off + (size_t)rr * p.ldc + c0 + 4 * hl;
                __stcs((float4*)(p.sgd_v + off), v);
                __stcs((float4*)(p.sgd_w + off), w);
                if (p.sgd_s != nullptr) {
                    __nv_bfloat162 lo = __floats2bfloat162_rn(w.x, w.y), hi = __floats2bfloat162_rn(w.z, w.w);
                    uint2 pk;
                    pk.x = *(uint32_t*)&lo;
                    pk.y = *(uint32_t*)&hi;
                    *(uint2*)(p.sgd_s + off) = pk;
                }
            }
        }
        epi_bar_sync();                                   // stage and slab buffer may be overwritten
        if (ok && threadIdx.x == 64 && j + 2 < BN / 64 && n0 + c0 + 128 < n_hi)
            upd_request_slab(mapW, mapV, slab_buf + (size_t)(j & 1) * UPD_SLAB_BYTES, &slab_bar[j & 1], n0 + c0 + 128, m0);
    }
    return ok;
}

// 16 consecutive output columns of one tile row, as bf16, into the staged tile (64-column slabs of 128 rows x 128 bytes in the
// 128-byte swizzle of the output tensor map).
__device__ __forceinline__ void stage_chunk16(const float (&f)[16], uint32_t row_s, uint32_t sw, int c0)
{
    uint32_t pk[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        __nv_bfloat162 t = __floats2bfloat162_rn(f[2 * j], f[2 * j + 1]);
        pk[j] = *(uint32_t*)&t;
    }
    const uint32_t slab = row_s + (uint32_t)(c0 >> 6) * 16384u, j0 = (uint32_t)(c0 & 63) >> 3;
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slab + ((j0 ^ sw) << 4)), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slab + (((j0 + 1u) ^ sw) << 4)), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]) : "memory");
}

// Data-gradient epilogue, staged output: the ReLU-mask row of this thread (BN bf16 values of the layer's input at the thread's
// pixel) is fetched into registers before the accumulator is waited for, so that the loads' latency hides behind the main
// loop (read per 16-column chunk inside the epilogue it cost 0.5 - 0.8 us per chunk, 3 - 4 us per 128-wide tile).
// (256-wide tiles keep a window of 128 columns in registers: store_row refills a slot with the values 128 columns further on
// as soon as it has used it, seven chunks ahead of their use)
template <int BN> struct MaskRow { static constexpr int SLOTS = (BN < 128 ? BN : 128) / 8; };
template <int MODE, int BN>
__device__ __forceinline__ bool prefetch_mask_row(const UmmaParams& p, bool row_ok, size_t row_off, int n0, int n_hi, uint4* refq)
{
    if (!(MODE == MODE_DGRAD && p.tma_out && p.epi == UEPI_MASK && p.ref != nullptr)) return false;
    const uint4* rp = (const uint4*)(p.ref + row_off + n0);
#pragma unroll
    for (int j = 0; j < MaskRow<BN>::SLOTS; ++j) refq[j] = (row_ok && n0 + 8 * j < n_hi) ? __ldg(rp + j) : make_uint4(0u, 0u, 0u, 0u);
    return true;
}

// Epilogue of one accumulator row: reads BN columns of this warp's TMEM lane quadrant (16 at a time) and
// writes them as raw split partial sums, or with bias + ReLU / the ReLU mask applied, as float or bf16.
template <int MODE, int BN>
__device__ __forceinline__ void store_row(const UmmaParams& p, uint32_t taddr, bool row_ok, size_t row_off, int n0, int n_hi,
                                          int split, const float* s_bias, uint8_t* stage = nullptr, int row = 0, const uint4* refq = nullptr)
{
    if (MODE == MODE_DGRAD && stage != nullptr && refq != nullptr) {
        // Staged data-gradient tile whose ReLU-mask row (BN bf16 values of the layer input) the caller fetched into registers
        // while the main loop ran: nothing in this loop waits for global memory.  Fully unrolled, so that refq[] stays in
        // registers.
        const uint32_t row_s = smem_u32(stage) + (uint32_t)row * 128u;
        const uint32_t sw = (uint32_t)(row & 7);
        constexpr int SLOTS = MaskRow<BN>::SLOTS;
        uint4* rq = const_cast<uint4*>(refq);
        const uint4* rp = (const uint4*)(p.ref + row_off + n0);
#pragma unroll
        for (int c0 = 0; c0 < BN; c0 += 32) {
            uint32_t v[2][16];
            tmem_ld16(taddr + c0, v[0]);     // warp-collective; two loads per wait
            tmem_ld16(taddr + c0 + 16, v[1]);
            tmem_ld_wait();
            if (n0 + c0 >= n_hi) continue;            // (uniform: whole 64-column slabs)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c = c0 + 16 * h;
                const uint4 r0 = rq[(c / 8) % SLOTS], r1 = rq[(c / 8 + 1) % SLOTS];
                if (c + 128 < BN) {                       // refill the two slots for the chunk 128 columns on
                    const bool more = row_ok && n0 + c + 128 < n_hi;
                    rq[(c / 8) % SLOTS] = more ? __ldg(rp + (c + 128) / 8) : make_uint4(0u, 0u, 0u, 0u);
                    rq[(c / 8 + 1) % SLOTS] = more ? __ldg(rp + (c + 128) / 8 + 1) : make_uint4(0u, 0u, 0u, 0u);
                }
                const __nv_bfloat16* rb0 = (const __nv_bfloat16*)&r0;
                const __nv_bfloat16* rb1 = (const __nv_bfloat16*)&r1;
                float f[16];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    f[j] = (__bfloat162float(rb0[j]) > 0.f) ? __uint_as_float(v[h][j]) : 0.f;
                    f[8 + j] = (__bfloat162float(rb1[j]) > 0.f) ? __uint_as_float(v[h][8 + j]) : 0.f;
                }
                stage_chunk16(f, row_s, sw, c);
            }
        }
        return;
    }
    if (MODE != MODE_WGRAD && stage != nullptr) {
        // Staged bf16 tile for the TMA store (the planner only selects it for unsplit bf16 outputs whose columns end on
        // 64-column slabs): every decision is taken once, outside the loop -- an epilogue warp runs alone on its
        // scheduler, so every branch and every dependent instruction in the loop costs its full latency.
        const bool bias_act = p.epi == UEPI_BIAS_ACT, relu = p.relu != 0;
        const __nv_bfloat16* refrow = (p.epi == UEPI_MASK && p.ref != nullptr && row_ok) ? p.ref + row_off + n0 : nullptr;
        const uint32_t bias_s = smem_u32(s_bias);
        const uint32_t row_s = smem_u32(stage) + (uint32_t)row * 128u;
        const uint32_t sw = (uint32_t)(row & 7);
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
            uint32_t v[2][16];
            tmem_ld16(taddr + c0, v[0]);     // warp-collective; two loads per wait
            tmem_ld16(taddr + c0 + 16, v[1]);
            tmem_ld_wait();
            if (n0 + c0 >= n_hi) continue;            // (uniform: whole 64-column slabs)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c = c0 + 16 * h;
                float f[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) f[j] = __uint_as_float(v[h][j]);
                if (bias_act) {
#pragma unroll
                    for (int j4 = 0; j4 < 4; ++j4) {
                        float b0, b1, b2, b3;
                        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(b0), "=f"(b1), "=f"(b2), "=f"(b3) : "r"(bias_s + (uint32_t)(c + 4 * j4) * 4u));
                        f[4 * j4] += b0; f[4 * j4 + 1] += b1; f[4 * j4 + 2] += b2; f[4 * j4 + 3] += b3;
                    }
                    if (relu) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) f[j] = f[j] > 0.f ? f[j] : 0.f;     // (NaN -> 0, as the reference path)
                    }
                } else if (refrow != nullptr) {
                    const uint4 r0 = *(const uint4*)(refrow + c), r1 = *(const uint4*)(refrow + c + 8);
                    const __nv_bfloat16* rb0 = (const __nv_bfloat16*)&r0;
                    const __nv_bfloat16* rb1 = (const __nv_bfloat16*)&r1;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (!(__bfloat162float(rb0[j]) > 0.f)) f[j] = 0.f;
                        if (!(__bfloat162float(rb1[j]) > 0.f)) f[8 + j] = 0.f;
                    }
                }
                stage_chunk16(f, row_s, sw, c);
            }
        }
        return;
    }
    const bool raw_partials = MODE != MODE_WGRAD && p.splits > 1;
    if (raw_partials || p.epi == UEPI_F32) {
        // Float rows without any arithmetic: the split partial sums of a forward / data-gradient op, or a weight-gradient
        // tile (straight into the gradient or into a split copy).  Destination and vector-store decision taken once.
        float* dst = raw_partials ? p.part + (size_t)split * p.split_stride + row_off + n0 : (float*)p.out + row_off + n0;
        const bool vec = raw_partials ? ((p.n_total & 3) == 0 && (n0 & 3) == 0)
                                      : ((p.ldc & 3) == 0 && (n0 & 3) == 0 && ((((size_t)p.split_stride) & 3) == 0) && ((p.w_cols & 3) == 0 || MODE != MODE_WGRAD));
        // (32-byte stores where the row allows: a thread writes a row of its own, so every store instruction of a warp
        // touches 32 different lines, and a 16-byte store leaves half of its 32-byte sector to a second instruction)
        const bool vec8 = vec && ((((uintptr_t)dst) & 31) == 0);
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 16) {
            uint32_t v[16];
            tmem_ld16(taddr + c0, v);     // warp-collective: executed by all lanes regardless of row_ok
            tmem_ld_wait();
            if (!row_ok || n0 + c0 >= n_hi) continue;
            if (vec8 && n0 + c0 + 16 <= n_hi) {
#pragma unroll
                for (int j = 0; j < 2; ++j)
                    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + c0 + 8 * j), "r"(v[8 * j]), "r"(v[8 * j + 1]),
                                 "r"(v[8 * j + 2]), "r"(v[8 * j + 3]), "r"(v[8 * j + 4]), "r"(v[8 * j + 5]), "r"(v[8 * j + 6]), "r"(v[8 * j + 7]) : "memory");
            } else if (vec && n0 + c0 + 16 <= n_hi) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    ((float4*)(dst + c0))[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (n0 + c0 + j < n_hi) dst[c0 + j] = __uint_as_float(v[j]);
            }
        }
        return;
    }
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += 16) {
        uint32_t v[16];
        tmem_ld16(taddr + c0, v);     // warp-collective: executed by all lanes regardless of row_ok
        tmem_ld_wait();
        if (!row_ok || n0 + c0 >= n_hi) continue;
        float f[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) f[j] = __uint_as_float(v[j]);
        const int ncol = n0 + c0;
        const bool full16 = ncol + 16 <= n_hi;
        if (MODE != MODE_WGRAD && p.splits > 1) {
            // split reduction: raw partial sums; bias / ReLU / mask / rounding happen in the reduce kernel
            float* op = p.part + (size_t)split * p.split_stride + row_off + ncol;   // ldc == n_total in these modes
            if (full16 && ((p.n_total & 3) == 0) && ((ncol & 3) == 0)) {
#pragma unroll
                for (int j = 0; j < 4; ++j) ((float4*)op)[j] = make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]);
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (ncol + j < n_hi) op[j] = f[j];
            }
            continue;
        }
        if (p.epi == UEPI_BIAS_ACT) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                f[j] += s_bias[c0 + j];
                if (p.relu && !(f[j] > 0.f)) f[j] = 0.f;
            }
        } else if (p.epi == UEPI_MASK && p.ref != nullptr) {
            const __nv_bfloat16* rp = p.ref + row_off + ncol;
            if (full16 && ((p.ldc & 7) == 0) && ((ncol & 7) == 0)) {
                uint4 r0 = *(const uint4*)rp, r1 = *(const uint4*)(rp + 8);
                const __nv_bfloat16* rb0 = (const __nv_bfloat16*)&r0;
                const __nv_bfloat16* rb1 = (const __nv_bfloat16*)&r1;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (!(__bfloat162float(rb0[j]) > 0.f)) f[j] = 0.f;
                    if (!(__bfloat162float(rb1[j]) > 0.f)) f[8 + j] = 0.f;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (ncol + j < n_hi && !(__bfloat162float(rp[j]) > 0.f)) f[j] = 0.f;
            }
        }
        if (p.epi == UEPI_F32 || p.out_f32) {
            float* op = (float*)p.out + row_off + ncol;
            if (full16 && ((p.ldc & 3) == 0) && ((ncol & 3) == 0) && ((((size_t)p.split_stride) & 3) == 0) && ((p.w_cols & 3) == 0 || MODE != MODE_WGRAD)) {
#pragma unroll
                for (int j = 0; j < 4; ++j) ((float4*)op)[j] = make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]);
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (ncol + j < n_hi) op[j] = f[j];
            }
        } else {
            __nv_bfloat16* op = (__nv_bfloat16*)p.out + row_off + ncol;
            if (full16 && ((p.ldc & 7) == 0) && ((ncol & 7) == 0)) {
                uint32_t pk[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    __nv_bfloat162 t = __floats2bfloat162_rn(f[2 * j], f[2 * j + 1]);
                    pk[j] = *(uint32_t*)&t;
                }
                if (stage != nullptr) {
                    // TMA-store staging: 64-column slabs of 128 rows x 128 bytes in the 128-byte swizzle of the tensor map
                    uint8_t* slab = stage + (c0 >> 6) * 16384 + row * 128;
                    const int j0 = (c0 & 63) >> 3;
                    *(uint4*)(slab + ((j0 ^ (row & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    *(uint4*)(slab + (((j0 + 1) ^ (row & 7)) << 4)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                } else {
                    ((uint4*)op)[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    ((uint4*)op)[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                }
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (ncol + j < n_hi) op[j] = __float2bfloat16_rn(f[j]);
            }
        }
    }
}

// 2x2 max-pool of the output tile staged for the TMA store (64-column slabs of 128 rows x 128 bytes, 16-byte chunks
// XOR-swizzled by row % 8; tile row = wi + bw * (hi + bh * ni), or wi + bw * (ni + bn * hi) in the halo kernel's order,
// with bw, bh even, so every pooling window lies inside the tile).  One task = one pooled pixel x 8 channels: four 16-byte shared-memory reads, one 16-byte store of the
// maxima and one 8-byte store of the argmax positions (dh*2+dw, the first maximum wins: the same rule and the same
// bf16 inputs as the stand-alone pooling kernel, so the bytes are identical).  Called by the 128 epilogue threads.
template <int BN>
__device__ __forceinline__ void pool_from_stage(const UmmaParams& p, const uint8_t* stage, int t128, int n0, int n_hi, int pw0, int ph0, int pn0)
{
    constexpr int CH = BN / 8;
    const int wb = p.bw / 2, hb = p.bh / 2, Ho = p.H / 2, Wo = p.W / 2;
    // tile row of pixel (wi, hi, ni) = wi + h_step * hi + n_step * ni
    const int h_step = p.hn_order ? p.bw * p.bn : p.bw, n_step = p.hn_order ? p.bw : p.bw * p.bh;
    for (int t = t128; t < 32 * CH; t += 128) {
        const int c = t % CH, pr = t / CH;
        const int pq = fast_div(pr, p.rcp_wb), nl = fast_div(pr, p.rcp_wbhb);
        const int wl = pr - pq * wb, hl = pq - nl * hb;
        const int w = pw0 + 2 * wl, h = ph0 + 2 * hl, n = pn0 + nl, ncol = n0 + 8 * c;
        if (w >= p.W || h >= p.H || n >= p.N || ncol >= n_hi) continue;
        const int r00 = 2 * wl + h_step * 2 * hl + n_step * nl;
        const uint8_t* slab = stage + (c >> 3) * 16384;
        const int cj = c & 7;
        uint4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int r = r00 + (j & 1) + (j >> 1) * h_step;
            v[j] = *(const uint4*)(slab + r * 128 + ((cj ^ (r & 7)) << 4));
        }
        uint4 outv;
        uint2 outi;
        __nv_bfloat16* ov = (__nv_bfloat16*)&outv;
        uint8_t* oi = (uint8_t*)&outi;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            __nv_bfloat16 bestv = ((const __nv_bfloat16*)&v[0])[k];
            float best = __bfloat162float(bestv);
            int bi = 0;
#pragma unroll
            for (int j = 1; j < 4; ++j) {
                const __nv_bfloat16 cand = ((const __nv_bfloat16*)&v[j])[k];
                const float f = __bfloat162float(cand);
                if (f > best) { best = f; bi = j; bestv = cand; }
            }
            ov[k] = bestv;
            oi[k] = (uint8_t)bi;
        }
        const size_t o = (((size_t)n * Ho + (h >> 1)) * Wo + (w >> 1)) * (size_t)p.ldc + ncol;
        *(uint4*)(p.pool_out + o) = outv;
        *(uint2*)(p.pool_idx + o) = outi;
    }
}

// ------------------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------------------
template <int MODE, int BN>
__global__ void __launch_bounds__(UMMA_THREADS, 1)
umma_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, const __grid_constant__ CUtensorMap mapC,
            const __grid_constant__ CUtensorMap mapD, const UmmaParams p)
{
    using C = Cfg<MODE, BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int STAGES = p.stages;
    uint8_t* ctrl = smem + STAGES * C::STAGE_BYTES;
    uint64_t* full = (uint64_t*)ctrl;                 // [MAX_STAGES]
    uint64_t* empty = full + MAX_STAGES;              // [MAX_STAGES]
    uint64_t* acc_full = empty + MAX_STAGES;          // [1]
    uint32_t* tmem_slot = (uint32_t*)(acc_full + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    uint64_t* slab_bar = (uint64_t*)(ctrl + 256);     // [2] WGRAD with the update folded in: parameter slabs landed
    float* s_bias = (float*)(ctrl + 512);             // [BN]
    uint8_t* slab_buf = ctrl + CTRL_BYTES;            // ... and the two slab buffers (only allocated for such launches)

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const unsigned cta_lin = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
#ifdef SB_CTA_TIMING
    unsigned long long* tlog = (p.timing != nullptr && cta_lin < 1024) ? p.timing + 16ull * cta_lin : nullptr;
#endif
    (void)cta_lin;
    SB_TLOG(threadIdx.x == 0, 0, globaltimer_ns());
    SB_TRACE_BEGIN();
    SB_TLOG(threadIdx.x == 0, 6, clock64());

    // ---- tile coordinates ---------------------------------------------------------------------
    int tap_fixed = 0, split = 0;
    int m_idx = blockIdx.x, n_idx = blockIdx.y;
    int n0, n_hi;       // first output column of this tile and one past the last valid column
    if (MODE == MODE_WGRAD) {
        tap_fixed = (blockIdx.z / p.splits) * p.tap_group;   // first tap of this CTA's group
        split = blockIdx.z % p.splits;
        n0 = n_idx * BN;
        n_hi = p.n_total;                                     // tap_group = 3: 3 x Cin (the taps' columns are adjacent)
        if (p.tap_group == 2) n_hi = min(p.n_total, (9 - tap_fixed) * p.w_cols);   // the last pair of taps has one member
    } else {
        if (p.shards == 1) {
            n0 = n_idx * BN;
            n_hi = p.n_total;
        } else {
            const int sh = n_idx / p.tiles_per_shard, t = n_idx % p.tiles_per_shard;
            const int lo = (int)(((long)sh * p.n_total) / p.shards), hi = (int)(((long)(sh + 1) * p.n_total) / p.shards);
            n0 = lo + t * BN;
            n_hi = hi;
        }
        if (n0 >= n_hi) return;   // uniform over the CTA, before any barrier or TMEM allocation
    }
    // FWD/DGRAD: the M tile is one pixel box; WGRAD: the M tile is 128 gradient rows of one shard
    int pw0 = 0, ph0 = 0, pn0 = 0, m0 = 0, m_hi = 0;
    if (MODE == MODE_WGRAD) {
        const int sh = m_idx / p.m_tiles_per_shard, t = m_idx % p.m_tiles_per_shard;
        const int lo = (int)(((long)sh * p.m_total) / p.m_shards), hi = (int)(((long)(sh + 1) * p.m_total) / p.m_shards);
        m0 = lo + t * 128;
        m_hi = hi;
        if (m0 >= m_hi) return;
    } else {
        const int q1 = fast_div_exact(m_idx, p.rcp_tiles_w, p.tiles_w), q2 = fast_div_exact(m_idx, p.rcp_tiles_wh, p.tiles_w * p.tiles_h);
        pw0 = (m_idx - q1 * p.tiles_w) * p.bw;
        ph0 = (q1 - q2 * p.tiles_h) * p.bh;
        pn0 = q2 * p.bn;
    }
    if (MODE != MODE_WGRAD) split = blockIdx.z;
    // k-iterations of this CTA: a contiguous range of the reduction
    const int k_begin = split * p.chunks_per_split;
    const int k_end = min(k_begin + p.chunks_per_split, p.total_chunks);
    const int n_iters = k_end - k_begin;
    // (tap groups {3,4,5} and {4,5} both start with a tap every CTA grid has exactly once per M tile and split)
    const bool do_bias = MODE == MODE_WGRAD && p.bias_fused && n_idx == 0 && tap_fixed == (p.ntaps == 9 ? (p.tap_group == 3 ? 3 : 4) : 0);

    // Operand loads of the next k-iteration into ring slot `s` (executed by the producer thread, iterations in
    // order).  The iteration's coordinates are carried in counters, so the issue path has no integer division.
    int ld_a = 0, ld_b = 0, ld_c = 0;   // WGRAD: pixel-box indices (w, h, n); FWD/DGRAD: (k-chunk, tap, unused)
    if (k_begin != 0) {      // (an unsplit reduction starts at zero: no division on that path)
        if (MODE == MODE_WGRAD) {
            ld_a = k_begin % p.tiles_w; ld_b = (k_begin / p.tiles_w) % p.tiles_h; ld_c = k_begin / (p.tiles_w * p.tiles_h);
        } else {
            ld_a = k_begin % p.kchunks; ld_b = k_begin / p.kchunks;
        }
    }
    const int wg_dr = p.ntaps == 9 ? tap_fixed / 3 - 1 : 0, wg_ds = p.ntaps == 9 ? tap_fixed % 3 - 1 : 0;
    // WGRAD with at most 64 gradient rows left in this tile: the second 64-row box of A would be all padding, so it
    // is not fetched (accumulator rows 64.. then hold garbage that is never stored; MMA rows are independent)
    const int a_boxes = (MODE == MODE_WGRAD && m0 + 64 >= m_hi) ? 1 : 2;
    // filter-column variant of the 64-input-channel weight gradient (BN = 192, hn_order): bytes between image rows of the
    // activation box, and the box's size with its two halo rows
    const uint32_t col_row_step = (uint32_t)(p.bw * p.bn) * 128u, col_box_bytes = (uint32_t)(p.bh + 2) * col_row_step;
    // (executed by the whole producer warp in lock-step: every value below is the same in all lanes, the lane with
    // el != 0 issues; ring slot and smem offset are carried in counters)
    int ld_s = 0;
    uint32_t ld_off = 0;
    const uint32_t smem0 = smem_u32(smem), full0 = smem_u32(&full[0]);
    // part 0: both operands; FWD / DGRAD only: 1 = the barrier's byte count and the weight operand, 2 = the activation operand
    auto issue_loads = [&](uint32_t el, int part = 0) {
        const uint32_t sa = smem0 + ld_off, sb = sa + A_STAGE_BYTES, bar = full0 + 8u * (uint32_t)ld_s;
        if (part != 2)
        mbar_expect_tx_el(bar, (MODE == MODE_WGRAD && BN == 192 && p.hn_order ? (uint32_t)A_STAGE_BYTES + col_box_bytes : (uint32_t)C::STAGE_BYTES) -
                                   (a_boxes == 2 ? 0u : 8192u), el);
        if (MODE == MODE_WGRAD) {
            // pixel chunk -> box origin; A = dy (two 64-channel boxes), B = shifted activations
            const int cw = ld_a * p.bw, ch = ld_b * p.bh, cn = ld_c * p.bn;
            if (BN == 192 && p.hn_order) {
                // one filter COLUMN: tensor maps with the dimensions listed as (c, w, n, h); one activation box with an image row
                // of halo above and below serves the three taps (the three 64-column panels of B are windows into it, see below)
                tma_load_4d_el(&mapA, sa, bar, m0, cw, cn, ch, el);
                if (a_boxes == 2) tma_load_4d_el(&mapA, sa + 8192, bar, m0 + 64, cw, cn, ch, el);
                tma_load_4d_el(&mapB, sb, bar, 0, cw + tap_fixed / 3 - 1, cn, ch - 1, el);
            } else {
            tma_load_4d_el(&mapA, sa, bar, m0, cw, ch, cn, el);
            if (a_boxes == 2) tma_load_4d_el(&mapA, sa + 8192, bar, m0 + 64, cw, ch, cn, el);
            if (BN == 192) {
                // one filter row: the three taps' activation boxes are the same pixels shifted by -1, 0, +1 in w
#pragma unroll
                for (int j = 0; j < 3; ++j) tma_load_4d_el(&mapB, sb + j * 8192, bar, 0, cw + j - 1, ch + wg_dr, cn, el);
            } else if (BN == 256 && p.tap_group == 2) {
                // two adjacent taps of a 128-input-channel layer: boxes 0, 1 = channels 0-63, 64-127 of tap t, boxes 2, 3 of
                // tap t + 1 (tap 9 does not exist: its rows lie outside the image and read as zeros, its columns are not stored)
                const int t1 = tap_fixed + 1, dr1 = t1 / 3 - 1, ds1 = t1 % 3 - 1;
                tma_load_4d_el(&mapB, sb, bar, 0, cw + wg_ds, ch + wg_dr, cn, el);
                tma_load_4d_el(&mapB, sb + 8192, bar, 64, cw + wg_ds, ch + wg_dr, cn, el);
                tma_load_4d_el(&mapB, sb + 16384, bar, 0, cw + ds1, ch + dr1, cn, el);
                tma_load_4d_el(&mapB, sb + 24576, bar, 64, cw + ds1, ch + dr1, cn, el);
            } else {
#pragma unroll
                for (int j = 0; j < BN / 64; ++j) tma_load_4d_el(&mapB, sb + j * 8192, bar, n0 + 64 * j, cw + wg_ds, ch + wg_dr, cn, el);
            }
            }
            if (++ld_a == p.tiles_w) { ld_a = 0; if (++ld_b == p.tiles_h) { ld_b = 0; ++ld_c; } }
        } else {
            const int kc = ld_a, tap = ld_b;
            int dr = 0, ds = 0;
            if (p.ntaps == 9) { const int r3 = tap >= 6 ? 2 : (tap >= 3 ? 1 : 0); dr = r3 - 1; ds = tap - 3 * r3 - 1; }
            if (MODE == MODE_DGRAD) { dr = -dr; ds = -ds; }
            if (part != 1) tma_load_4d_el(&mapA, sa, bar, kc * 64, pw0 + ds, ph0 + dr, pn0, el);
            if (part == 2) {
            } else if (MODE == MODE_FWD) {
                tma_load_4d_el(&mapB, sb, bar, tap * p.w_cols + kc * 64, n0, 0, 0, el);
            } else {
#pragma unroll
                for (int j = 0; j < BN / 64; ++j) tma_load_4d_el(&mapB, sb + j * 8192, bar, tap * p.w_cols + n0 + 64 * j, kc * 64, 0, 0, el);
            }
            if (++ld_a == p.kchunks) { ld_a = 0; ++ld_b; }
        }
        ++ld_s; ld_off += (uint32_t)C::STAGE_BYTES;
        if (ld_s == STAGES) { ld_s = 0; ld_off = 0; }
    };
    const int preloaded = n_iters < STAGES ? n_iters : STAGES;

    // ---- one-time setup -----------------------------------------------------------------------
    // (programmatic dependent launch: everything up to pdl_wait() touches only shared memory and TMEM, so it
    // may run while the kernel this one depends on is still finishing)
    uint32_t prod_el = 0;
    if (warp == 0) {
        if (lane == 0) {
            // a stage is released by the MMA commit, plus one arrival per epilogue warp in the CTAs that also sum dy
            for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], do_bias ? 5u : 1u); }
            mbar_init(acc_full, 1);
            if (MODE == MODE_WGRAD && p.sgd_w != nullptr) { mbar_init(&slab_bar[0], 1); mbar_init(&slab_bar[1], 1); }
            *abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            SB_TLOG(true, 8, clock64());    // barriers initialised
        }
        __syncwarp();
        prod_el = elect_one() ? 1u : 0u;
        if (MODE != MODE_WGRAD && p.w_first) {
            // the weights are not the predecessor kernel's output: their first ring-full is on its way while that kernel finishes
            const int a0 = ld_a, b0 = ld_b;
            for (int it = 0; it < preloaded; ++it) issue_loads(prod_el, 1);
            ld_a = a0; ld_b = b0; ld_s = 0; ld_off = 0;
        }
        pdl_wait();
        pdl_trigger();
        SB_TRACE_STAMP(trace_a);
        SB_TLOG(lane == 0, 9, clock64());    // predecessor kernel complete
        // The first ring-full of loads needs nothing but the barriers just initialised: start them now, so that
        // their latency overlaps the TMEM allocation and the rest of the set-up.
        for (int it = 0; it < preloaded; ++it) issue_loads(prod_el, (MODE != MODE_WGRAD && p.w_first) ? 2 : 0);
        SB_TLOG(lane == 0, 10, clock64());   // first ring of loads issued
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, C::TMEM_COLS);
        tmem_relinquish();
        SB_TLOG(lane == 0, 11, clock64());   // TMEM allocated
    }
    if (warp != 0) pdl_wait();   // every thread that will touch global memory waits for the predecessor kernel
    if (MODE == MODE_FWD && p.epi == UEPI_BIAS_ACT && warp >= 2) {
        for (int c = threadIdx.x - 64; c < BN; c += 128) s_bias[c] = (n0 + c < n_hi) ? p.bias[n0 + c] : 0.f;
    }
    SB_TLOG(threadIdx.x == 64, 12, clock64());   // bias staged
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    SB_TLOG(threadIdx.x == 0, 1, clock64());   // set-up done
    SB_TRACE_STAMP(trace_b);

    if (warp == 0) {
        // =========================== TMA producer ===============================================
        // the whole warp in lock-step; slot `ws` is free once the MMAs that read it have completed
        // Rings of four or more stages are refilled two slots per round: both releases are polled together (two
        // independent barrier reads in flight) and the loads of both iterations go out back to back.  Taken one slot
        // at a time, the wait -> issue chain of this warp, not the operand bytes, set the pace of the main loop
        // (measured with the loads switched off: the same time per iteration).  Shallow rings keep the one-slot step: a
        // producer that waits for two free slots out of two or three would stall the MMA warp.
        int ws = 0;
        uint32_t wph = 0;
        const int batch = STAGES >= 4 ? 2 : 1;
        bool got = true;
        for (int it = preloaded; it < n_iters;) {
            const int nb = (batch == 2 && it + 1 < n_iters) ? 2 : 1;
            const int s2 = ws + 1 == STAGES ? 0 : ws + 1;
            const uint32_t p2 = s2 == 0 ? wph ^ 1u : wph;
            const bool w1 = mbar_try_wait(&empty[ws], wph), w2 = nb == 2 ? mbar_try_wait(&empty[s2], p2) : true;
            if (!__all_sync(0xffffffffu, (w1 && w2) ? 1 : 0)) {
                got = __all_sync(0xffffffffu, (mbar_wait(&empty[ws], wph) && (nb == 1 || mbar_wait(&empty[s2], p2))) ? 1 : 0) != 0;
                if (!got) break;
            }
            issue_loads(prod_el);
            if (nb == 2) issue_loads(prod_el);
            if (nb == 2) { ws = s2 + 1; wph = p2; } else { ws = ws + 1; }
            if (ws == STAGES) { ws = 0; wph ^= 1u; }
            it += nb;
        }
        if (!got && lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_TMA); }
        SB_TRACE_STAMP(trace_c);
        __syncwarp();
    } else if (warp == 1) {
        // =========================== MMA issuer =================================================
        // The whole warp walks the ring in lock-step (barrier waits, descriptor words and ring counters are the same
        // in every lane, so they live in uniform registers); one elected lane issues the MMAs and the commits.
        constexpr uint32_t idesc = make_idesc(BN, MODE == MODE_WGRAD, MODE != MODE_FWD);
        const uint32_t elected = elect_one() ? 1u : 0u;
        const uint32_t sa0 = smem_u32(smem);
        // K-major: 16 elements = 32 bytes along the row; MN-major: 16 k-rows = 2048 bytes
        const uint64_t dA0 = (MODE == MODE_WGRAD) ? make_desc(sa0, 8192) : make_desc(sa0, 16);
        // (filter-column weight gradient: the three 64-column panels of B are the same activation box read one image row
        // apart -- tap row r starts r * bw * bn rows into it, a whole number of 8-row swizzle groups)
        const uint64_t dB0 = (MODE == MODE_FWD) ? make_desc(sa0 + A_STAGE_BYTES, 16)
                                                : make_desc(sa0 + A_STAGE_BYTES, (MODE == MODE_WGRAD && BN == 192 && p.hn_order) ? col_row_step : 8192u);
        const uint32_t a_hi = (uint32_t)(dA0 >> 32), b_hi = (uint32_t)(dB0 >> 32);
        const uint32_t a_lo0 = (uint32_t)dA0, b_lo0 = (uint32_t)dB0;
        constexpr uint32_t A_STEP = ((MODE == MODE_WGRAD) ? 2048u : 32u) >> 4, B_STEP = ((MODE == MODE_FWD) ? 32u : 2048u) >> 4;
        constexpr uint32_t STAGE16 = (uint32_t)C::STAGE_BYTES >> 4;     // the address field counts 16-byte units
        int s = 0;
        uint32_t ph = 0, off = 0;
        bool ok = true;
        // two ring slots per round where the ring is deep enough (see the producer): both full barriers are polled together
        // and the eight MMAs go out back to back
        const int batch = STAGES >= 4 ? 2 : 1;
        for (int it = 0; it < n_iters;) {
            const int nb = (batch == 2 && it + 1 < n_iters) ? 2 : 1;
            const int s2 = s + 1 == STAGES ? 0 : s + 1;
            const uint32_t p2 = s2 == 0 ? ph ^ 1u : ph, off2 = s2 == 0 ? 0u : off + STAGE16;
            const bool w1 = mbar_try_wait(&full[s], ph), w2 = nb == 2 ? mbar_try_wait(&full[s2], p2) : true;
            if (!__all_sync(0xffffffffu, w1 ? 1 : 0)) {
                ok = __all_sync(0xffffffffu, mbar_wait(&full[s], ph) ? 1 : 0) != 0;
                if (!ok) break;
            }
            SB_TLOG(lane == 0 && it == 0, 2, clock64());            // first operands landed
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                umma_bf16_lohi(tmem_base, a_lo0 + off + kk * A_STEP, a_hi, b_lo0 + off + kk * B_STEP, b_hi, idesc, (it > 0 || kk > 0) ? 1u : 0u, elected);
            if (elected) umma_commit(&empty[s]);      // stage reusable once these MMAs have read it
            if (nb == 2) {
                if (!__all_sync(0xffffffffu, w2 ? 1 : 0)) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&full[s2], p2) ? 1 : 0) != 0;
                    if (!ok) break;
                    tc_fence_after();
                }
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_bf16_lohi(tmem_base, a_lo0 + off2 + kk * A_STEP, a_hi, b_lo0 + off2 + kk * B_STEP, b_hi, idesc, 1u, elected);
                if (elected) umma_commit(&empty[s2]);
                s = s2; off = off2; ph = p2;
            }
            SB_TLOG(lane == 0 && it + nb >= n_iters, 3, clock64());  // last operands landed
            __syncwarp();
            ++s; off += STAGE16;
            if (s == STAGES) { s = 0; off = 0; ph ^= 1u; }
            it += nb;
        }
        if (!ok && lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_MMA); }
        if (ok && elected) umma_commit(acc_full);   // accumulator complete
        __syncwarp();
    } else {
        // =========================== epilogue ===================================================
        const int q = warp % 4;               // TMEM lane quadrant of this warp
        const int row = q * 32 + lane;        // accumulator row handled by this thread
        bool ok = true;
        // where this thread's accumulator row goes (computed while the main loop runs)
        bool row_ok;
        size_t row_off;
        if (MODE == MODE_WGRAD) {
            row_ok = (m0 + row) < m_hi;
            row_off = (size_t)split * p.split_stride + (size_t)(m0 + row) * p.ldc + (size_t)tap_fixed * p.w_cols;
            if (p.sgd_w != nullptr && threadIdx.x == 64) {
                // update folded in: the w and v boxes of the first two 64-column slabs are requested now
#pragma unroll
                for (int j = 0; j < 2; ++j)
                    if (j < BN / 64 && n0 + 64 * j < n_hi)
                        upd_request_slab(&mapC, &mapD, slab_buf + (size_t)j * UPD_SLAB_BYTES, &slab_bar[j], n0 + 64 * j, m0);
            }
        } else {
            const int r1 = fast_div(row, p.rcp_bw), ni = fast_div(row, p.rcp_bwbh);
            const int wi = row - r1 * p.bw, hi_ = r1 - ni * p.bh;
            const int w = pw0 + wi, h = ph0 + hi_, n = pn0 + ni;
            row_ok = w < p.W && h < p.H && n < p.N;
            row_off = (((size_t)n * p.H + h) * p.W + w) * p.ldc;
        }
        if (MODE == MODE_WGRAD && do_bias) {
            // Bias gradient: thread `row` sums dy[pixel, m0 + row] over this CTA's pixel chunks, reading the A
            // stage (64 pixel rows of 128 bytes per 64-channel box, 16-byte chunks XOR-swizzled by row % 8)
            // while the MMA consumes it; pixel order is fixed, so the sum is deterministic.
            float bsum = 0.f;
            const uint32_t box_off = (uint32_t)(row / 64) * 8192u, c = (uint32_t)(row % 64);
            for (int it = 0; it < n_iters && ok; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (uint32_t)((it / STAGES) & 1);
                if (lane == 0) ok = mbar_wait(&full[s], ph);
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                const uint8_t* sa = smem + s * C::STAGE_BYTES + box_off;
#pragma unroll 8
                for (uint32_t k = 0; k < 64; ++k) {
                    const uint32_t off = k * 128u + (((c >> 3) ^ (k & 7u)) << 4) + (c & 7u) * 2u;
                    bsum += __bfloat162float(*(const __nv_bfloat16*)(sa + off));
                }
                __syncwarp();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&empty[s])) : "memory");
            }
            if (ok && (m0 + row) < m_hi) {
                const size_t bo = (size_t)split * p.split_stride + p.bias_off + m0 + row;
                if (p.sgd_w != nullptr) {
                    const float vb = fmaf(p.sgd_mu, p.sgd_v[bo], bsum), wb = fmaf(-p.sgd_lr, vb, p.sgd_w[bo]);
                    p.sgd_v[bo] = vb;
                    p.sgd_w[bo] = wb;
                    if (p.sgd_s != nullptr) p.sgd_s[bo] = __float2bfloat16_rn(wb);
                } else {
                    ((float*)p.out)[bo] = bsum;
                }
            }
            if (!ok && lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_EPI); }
        }
        uint4 refq[MODE == MODE_DGRAD ? MaskRow<BN>::SLOTS : 1];
        const bool have_refq = prefetch_mask_row<MODE, BN>(p, row_ok, row_off, n0, n_hi, refq);
        if (lane == 0 && ok) ok = mbar_wait(acc_full, 0);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok && lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_EPI); }
        if (MODE == MODE_WGRAD && p.wg_sweep) {
            // (the four epilogue warps work on the tile together: all of them reach this barrier, also after a timeout)
            epi_bar_sync();
            if (!*abort_flag) {
                SB_TLOG(threadIdx.x == 64, 4, clock64());      // accumulator complete
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
                if (p.sgd_w != nullptr) {
                    if (!wgrad_sweep_update_epilogue<BN>(p, &mapC, &mapD, taddr, smem, slab_buf, slab_bar, row, m0, m_hi, n0, n_hi,
                                                         (size_t)split * p.split_stride + (size_t)m0 * p.ldc + (size_t)tap_fixed * p.w_cols + n0) && lane == 0) {
                        *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_EPI);
                    }
                } else if (BN == 192 && p.hn_order)      // slab j = tap row j of filter column tap_fixed / 3: gradient columns (3 j + column) * Cin ..
                    wgrad_sweep_epilogue<BN>(p, taddr, smem, row, m0, m_hi, n0, n_hi,
                                             (size_t)split * p.split_stride + (size_t)m0 * p.ldc + (size_t)(tap_fixed / 3) * p.w_cols, 3,
                                             STAGES * C::STAGE_BYTES >= 65536);
                else
                    wgrad_sweep_epilogue<BN>(p, taddr, smem, row, m0, m_hi, n0, n_hi,
                                             (size_t)split * p.split_stride + (size_t)m0 * p.ldc + (size_t)tap_fixed * p.w_cols + n0, 1,
                                             STAGES * C::STAGE_BYTES >= 65536);
            }
        } else if (ok) {
            SB_TLOG(threadIdx.x == 64, 4, clock64());      // accumulator complete
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
            // (the operand ring is idle once the accumulator is complete: its first bytes stage the output tile)
            store_row<MODE, BN>(p, taddr, row_ok, row_off, n0, n_hi, split, s_bias, (MODE != MODE_WGRAD && p.tma_out) ? smem : nullptr, row, have_refq ? refq : nullptr);
            if (MODE != MODE_WGRAD && p.tma_out) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
    }

    // ---- teardown: everyone meets here; TMEM is released on every path ----------------------------
    tc_fence_before();
    __syncthreads();
    if (MODE != MODE_WGRAD && p.tma_out && threadIdx.x == 64 && !*abort_flag) {
        // one 64-column slab per store: rows outside the image and columns outside the tensor are clipped
#pragma unroll
        for (int j = 0; j < BN / 64; ++j)
            if (n0 + 64 * j < n_hi) tma_store_4d(&mapC, smem_u32(smem) + j * 16384, n0 + 64 * j, pw0, ph0, pn0);
        tma_store_commit();
    }
    if (MODE == MODE_FWD && p.tma_out && p.pool_out != nullptr && warp >= 2 && !*abort_flag)
        pool_from_stage<BN>(p, smem, threadIdx.x - 64, n0, n_hi, pw0, ph0, pn0);     // reads the stage while the TMA stores read it too
    if (MODE != MODE_WGRAD && p.tma_out && threadIdx.x == 64 && !*abort_flag) tma_store_wait_read();   // shared memory may be released once the stores have read it; the writes complete with the grid
    SB_TLOG(threadIdx.x == 0, 5, clock64());   // epilogue done
    SB_TLOG(threadIdx.x == 0, 7, globaltimer_ns());
    SB_TRACE_END(0);
    if (*abort_flag) {
        // give copies that may still be in flight time to land before shared memory is released
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) { }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------
// The halo kernel (3x3 FWD / DGRAD): one activation fetch per filter column
// ------------------------------------------------------------------------------------------------
// In umma_kernel every (tap, 64-channel chunk) fetches its own 128-pixel activation box, so each activation pixel
// crosses L2 -> shared memory nine times per chunk and the main loop runs at the rate one SM pulls operands from L2.
// Here the three taps of one filter COLUMN (same shift in w, shifts -1, 0, +1 in h) share one fetch: the box carries
// bh + 2 image rows (a halo row above and below), it lies in shared memory as [h][n][w] rows of 128 bytes -- the
// tensor map lists the dimensions as (c, w, n, h) -- and tap row j = 0, 1, 2 reads the 128 tile rows that start
// j * bw * bn rows into it.  bw * bn is a multiple of 8, so that start is a whole number of 8-row swizzle groups and
// only the start address of the shared-memory descriptor moves.  Per 64-channel chunk the activations cross three
// times (once per shift in w) with (bh + 2) / bh of the box each, instead of nine times.  Zero padding, ragged tile
// edges and images past the batch are the TMA's out-of-bounds zero fill, as before.
//
// Two rings: activation halos (a_stages slots, one per (chunk, w shift) group, released after its three taps) and
// weight tiles (stages slots, one per tap, as in umma_kernel).  Warp roles, bounded waits, epilogues, the pooled
// output and programmatic dependent launch are those of umma_kernel; tile row = wi + bw * (ni + bn * hi).
constexpr int MAX_A_STAGES = 4;
template <int BN> struct HaloCfg {
    static constexpr int B_STAGE_BYTES = BN * 128;
    static constexpr int TMEM_COLS = BN;
    static constexpr int smem_bytes(int a_stages, int a_slot_bytes, int b_stages)
    {
        return a_stages * a_slot_bytes + b_stages * B_STAGE_BYTES + 1024 /*alignment slack*/ + CTRL_BYTES;
    }
};

template <int MODE, int BN>
__global__ void __launch_bounds__(UMMA_THREADS, 1)
umma_halo_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, const __grid_constant__ CUtensorMap mapC,
                 const UmmaParams p)
{
    static_assert(MODE == MODE_FWD || MODE == MODE_DGRAD, "halo kernel: forward and data gradient only");
    using C = HaloCfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int SA = p.a_stages, SB = p.stages;
    const uint32_t row_step = (uint32_t)(p.bw * p.bn) * 128u;          // bytes between halo rows (a multiple of 1024)
    const uint32_t a_slot = (uint32_t)(p.bh + 2) * row_step;
    uint8_t* b_ring = smem + (size_t)SA * a_slot;
    uint8_t* ctrl = b_ring + (size_t)SB * C::B_STAGE_BYTES;
    uint64_t* b_full = (uint64_t*)ctrl;               // [MAX_STAGES]
    uint64_t* b_empty = b_full + MAX_STAGES;          // [MAX_STAGES]
    uint64_t* a_full = b_empty + MAX_STAGES;          // [MAX_A_STAGES]
    uint64_t* a_empty = a_full + MAX_A_STAGES;        // [MAX_A_STAGES]
    uint64_t* acc_full = a_empty + MAX_A_STAGES;      // [1]
    uint32_t* tmem_slot = (uint32_t*)(acc_full + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    float* s_bias = (float*)(ctrl + 512);             // [BN]

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
#ifdef SB_CTA_TIMING
    const unsigned cta_lin = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
    unsigned long long* tlog = (p.timing != nullptr && cta_lin < 1024) ? p.timing + 16ull * cta_lin : nullptr;
#endif
    SB_TLOG(threadIdx.x == 0, 0, globaltimer_ns());
    SB_TRACE_BEGIN();
    SB_TLOG(threadIdx.x == 0, 6, clock64());

    // ---- tile coordinates ---------------------------------------------------------------------
    const int m_idx = blockIdx.x, split = blockIdx.z;
    const int n0 = blockIdx.y * BN, n_hi = p.n_total;
    if (n0 >= n_hi) return;   // uniform over the CTA, before any barrier or TMEM allocation
    const int q1 = fast_div_exact(m_idx, p.rcp_tiles_w, p.tiles_w), q2 = fast_div_exact(m_idx, p.rcp_tiles_wh, p.tiles_w * p.tiles_h);
    const int pw0 = (m_idx - q1 * p.tiles_w) * p.bw;
    const int ph0 = (q1 - q2 * p.tiles_h) * p.bh;
    const int pn0 = q2 * p.bn;
    // this CTA's groups: a contiguous range of the 3 * kchunks (chunk, w shift) groups
    const int g_begin = split * p.chunks_per_split;
    const int g_end = min(g_begin + p.chunks_per_split, p.total_chunks);
    const int n_groups = g_end - g_begin;

    // ---- producer state (whole warp in lock-step, elected issue: see umma_kernel) -----------------
    int ld_kc = 0, ld_dsi = 0;
    if (g_begin != 0) { ld_kc = g_begin / 3; ld_dsi = g_begin % 3; }
    int la_s = 0, lb_s = 0;
    uint32_t la_off = 0, lb_off = 0;
    const uint32_t smem0 = smem_u32(smem), bring0 = smem_u32(b_ring);
    const uint32_t afull0 = smem_u32(&a_full[0]), bfull0 = smem_u32(&b_full[0]);
    int dbg_a = 0, dbg_b = 0;
    (void)dbg_a; (void)dbg_b;
    auto issue_halo = [&](uint32_t el) {
        const uint32_t bar = afull0 + 8u * (uint32_t)la_s;
#ifdef SB_CTA_TIMING
        if ((p.dbg_skip & 1) && dbg_a++ >= SA) mbar_expect_tx_el(bar, 0u, el);
        else {
#endif
        mbar_expect_tx_el(bar, a_slot, el);
        tma_load_4d_el(&mapA, smem0 + la_off, bar, ld_kc * 64, pw0 + ld_dsi - 1, pn0, ph0 - 1, el);    // (c, w, n, h)
#ifdef SB_CTA_TIMING
        }
#endif
        ++la_s; la_off += a_slot;
        if (la_s == SA) { la_s = 0; la_off = 0; }
    };
    auto issue_weights = [&](int j, uint32_t el) {
        // halo row j and w shift ld_dsi - 1 belong to filter tap (r, s) = (j, dsi) in the forward pass and, the
        // shifts being mirrored, to (2 - j, 2 - dsi) in the data gradient
        const int tap = MODE == MODE_FWD ? 3 * j + ld_dsi : 3 * (2 - j) + (2 - ld_dsi);
        const uint32_t dst = bring0 + lb_off, bar = bfull0 + 8u * (uint32_t)lb_s;
#ifdef SB_CTA_TIMING
        if ((p.dbg_skip & 2) && dbg_b++ >= SB) mbar_expect_tx_el(bar, 0u, el);
        else {
#endif
        mbar_expect_tx_el(bar, (uint32_t)C::B_STAGE_BYTES, el);
        if (MODE == MODE_FWD) {
            tma_load_4d_el(&mapB, dst, bar, tap * p.w_cols + ld_kc * 64, n0, 0, 0, el);
        } else {
#pragma unroll
            for (int jj = 0; jj < BN / 64; ++jj) tma_load_4d_el(&mapB, dst + jj * 8192, bar, tap * p.w_cols + n0 + 64 * jj, ld_kc * 64, 0, 0, el);
        }
#ifdef SB_CTA_TIMING
        }
#endif
        ++lb_s; lb_off += (uint32_t)C::B_STAGE_BYTES;
        if (lb_s == SB) { lb_s = 0; lb_off = 0; }
    };
    auto next_group = [&]() { if (++ld_dsi == 3) { ld_dsi = 0; ++ld_kc; } };
    // whole groups that fit into both rings without waiting for a release
    int preloaded = SA < SB / 3 ? SA : SB / 3;
    if (preloaded > n_groups) preloaded = n_groups;

    // ---- one-time setup -----------------------------------------------------------------------
    uint32_t prod_el = 0;
    if (warp == 0) {
        if (lane == 0) {
            for (int s = 0; s < SB; ++s) { mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 1); }
            for (int s = 0; s < SA; ++s) { mbar_init(&a_full[s], 1); mbar_init(&a_empty[s], 1); }
            mbar_init(acc_full, 1);
            *abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
        prod_el = elect_one() ? 1u : 0u;
        if (p.w_first) {
            // the weights are not the predecessor kernel's output: the first groups' weight tiles are on their way while that
            // kernel finishes; the activation halos follow once it has
            const int kc0 = ld_kc, dsi0 = ld_dsi;
            for (int g = 0; g < preloaded; ++g) {
#pragma unroll
                for (int j = 0; j < 3; ++j) issue_weights(j, prod_el);
                next_group();
            }
            ld_kc = kc0; ld_dsi = dsi0;
        }
        pdl_wait();
        pdl_trigger();
        SB_TRACE_STAMP(trace_a);
        for (int g = 0; g < preloaded; ++g) {
            issue_halo(prod_el);
            if (!p.w_first) {
#pragma unroll
                for (int j = 0; j < 3; ++j) issue_weights(j, prod_el);
            }
            next_group();
        }
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, C::TMEM_COLS);
        tmem_relinquish();
    }
    if (warp != 0) pdl_wait();   // every thread that will touch global memory waits for the predecessor kernel
    if (MODE == MODE_FWD && p.epi == UEPI_BIAS_ACT && warp >= 2) {
        for (int c = threadIdx.x - 64; c < BN; c += 128) s_bias[c] = (n0 + c < n_hi) ? p.bias[n0 + c] : 0.f;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    SB_TLOG(threadIdx.x == 0, 1, clock64());   // set-up done
    SB_TRACE_STAMP(trace_b);

    if (warp == 0) {
        // =========================== TMA producer ===============================================
        // One group per round: the releases of its halo slot and of its three weight slots are polled together (four
        // independent barrier reads in flight instead of four waits one after the other), then the four copies are
        // issued.  A barrier that has not completed a phase yet reports the phase before its first as complete, so
        // the first pass over a ring waits for parity 1 and falls through; the parity flips at every wrap.  (Taken
        // tap by tap, with the wait parities recomputed by division, this loop was what set the pace of the whole
        // main loop: ~135 cycles per MMA against ~85 this way.)
        // (the preloaded groups took first uses only: preloaded <= SA and 3 * preloaded <= SB; a ring they filled exactly
        // has wrapped to slot 0, and its next use waits for the first release)
        uint32_t pa_par = (preloaded > 0 && la_s == 0) ? 0u : 1u, pb_par = (preloaded > 0 && lb_s == 0) ? 0u : 1u;
        bool ok = true;
        for (int g = preloaded; g < n_groups; ++g) {
            const int s1 = lb_s, s2 = s1 + 1 == SB ? 0 : s1 + 1, s3 = s2 + 1 == SB ? 0 : s2 + 1;
            const uint32_t p1 = pb_par, p2 = s2 == 0 ? p1 ^ 1u : p1, p3 = s3 == 0 ? p2 ^ 1u : p2;
            const bool w0 = mbar_try_wait(&a_empty[la_s], pa_par), w1 = mbar_try_wait(&b_empty[s1], p1),
                       w2 = mbar_try_wait(&b_empty[s2], p2), w3 = mbar_try_wait(&b_empty[s3], p3);
            if (!__all_sync(0xffffffffu, (w0 && w1 && w2 && w3) ? 1 : 0)) {
                ok = __all_sync(0xffffffffu, (mbar_wait(&a_empty[la_s], pa_par) && mbar_wait(&b_empty[s1], p1) &&
                                              mbar_wait(&b_empty[s2], p2) && mbar_wait(&b_empty[s3], p3)) ? 1 : 0) != 0;
                if (!ok) break;
            }
            const bool a_wraps = la_s + 1 == SA;
            issue_halo(prod_el);
            if (a_wraps) pa_par ^= 1u;
#pragma unroll
            for (int j = 0; j < 3; ++j) issue_weights(j, prod_el);
            pb_par = (s3 + 1 == SB) ? p3 ^ 1u : p3;
            next_group();
        }
        if (!ok && lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_TMA); }
        SB_TRACE_STAMP(trace_c);
        __syncwarp();
    } else if (warp == 1) {
        // =========================== MMA issuer =================================================
        constexpr uint32_t idesc = make_idesc(BN, 0, MODE != MODE_FWD);
        const uint32_t elected = elect_one() ? 1u : 0u;
        const uint64_t dA0 = make_desc(smem0, 16);
        const uint64_t dB0 = (MODE == MODE_FWD) ? make_desc(bring0, 16) : make_desc(bring0, 8192);
        const uint32_t a_hi = (uint32_t)(dA0 >> 32), b_hi = (uint32_t)(dB0 >> 32);
        const uint32_t a_lo0 = (uint32_t)dA0, b_lo0 = (uint32_t)dB0;
        constexpr uint32_t A_STEP = 32u >> 4, B_STEP = ((MODE == MODE_FWD) ? 32u : 2048u) >> 4;
        constexpr uint32_t BSTAGE16 = (uint32_t)C::B_STAGE_BYTES >> 4;     // the address field counts 16-byte units
        const uint32_t aslot16 = a_slot >> 4, rowstep16 = row_step >> 4;
        int sa = 0, sb_ = 0;
        uint32_t pha = 0, phb = 0, aoff = 0, boff = 0;
        bool ok = true;
        // One group per round: the four full barriers are polled together, then the twelve MMAs go out back to back
        // (a tap whose weights had not landed at the poll is waited for just before its own four).
        for (int g = 0; g < n_groups; ++g) {
            const int s1 = sb_, s2 = s1 + 1 == SB ? 0 : s1 + 1, s3 = s2 + 1 == SB ? 0 : s2 + 1;
            const uint32_t p1 = phb, p2 = s2 == 0 ? p1 ^ 1u : p1, p3 = s3 == 0 ? p2 ^ 1u : p2;
            const uint32_t o1 = boff, o2 = s2 == 0 ? 0u : o1 + BSTAGE16, o3 = s3 == 0 ? 0u : o2 + BSTAGE16;
            const bool w0 = mbar_try_wait(&a_full[sa], pha), w1 = mbar_try_wait(&b_full[s1], p1), w2 = mbar_try_wait(&b_full[s2], p2),
                       w3 = mbar_try_wait(&b_full[s3], p3);
            if (!__all_sync(0xffffffffu, (w0 && w1) ? 1 : 0)) {
                ok = __all_sync(0xffffffffu, (mbar_wait(&a_full[sa], pha) && mbar_wait(&b_full[s1], p1)) ? 1 : 0) != 0;
                if (!ok) break;
            }
            SB_TLOG(lane == 0 && g == 0, 2, clock64());                    // first operands landed
            tc_fence_after();
            const uint32_t alo = a_lo0 + aoff;
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                umma_bf16_lohi(tmem_base, alo + kk * A_STEP, a_hi, b_lo0 + o1 + kk * B_STEP, b_hi, idesc, (g > 0 || kk > 0) ? 1u : 0u, elected);
            if (elected) umma_commit(&b_empty[s1]);      // weight slot reusable once these MMAs have read it
            if (!__all_sync(0xffffffffu, w2 ? 1 : 0)) {
                ok = __all_sync(0xffffffffu, mbar_wait(&b_full[s2], p2) ? 1 : 0) != 0;
                if (!ok) break;
                tc_fence_after();
            }
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                umma_bf16_lohi(tmem_base, alo + rowstep16 + kk * A_STEP, a_hi, b_lo0 + o2 + kk * B_STEP, b_hi, idesc, 1u, elected);
            if (elected) umma_commit(&b_empty[s2]);
            if (!__all_sync(0xffffffffu, w3 ? 1 : 0)) {
                ok = __all_sync(0xffffffffu, mbar_wait(&b_full[s3], p3) ? 1 : 0) != 0;
                if (!ok) break;
                tc_fence_after();
            }
            SB_TLOG(lane == 0 && g == n_groups - 1, 3, clock64());         // last operands landed
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                umma_bf16_lohi(tmem_base, alo + 2 * rowstep16 + kk * A_STEP, a_hi, b_lo0 + o3 + kk * B_STEP, b_hi, idesc, 1u, elected);
            if (elected) {
                umma_commit(&b_empty[s3]);
                umma_commit(&a_empty[sa]);               // halo slot reusable once its three taps have read it
            }
            __syncwarp();
            sb_ = s3 + 1; boff = o3 + BSTAGE16; phb = p3;
            if (sb_ == SB) { sb_ = 0; boff = 0; phb ^= 1u; }
            ++sa; aoff += aslot16;
            if (sa == SA) { sa = 0; aoff = 0; pha ^= 1u; }
        }
        if (!ok && lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_MMA); }
        if (ok && elected) umma_commit(acc_full);   // accumulator complete
        __syncwarp();
    } else {
        // =========================== epilogue ===================================================
        const int q = warp % 4;               // TMEM lane quadrant of this warp
        const int row = q * 32 + lane;        // accumulator row handled by this thread
        // tile row = wi + bw * (ni + bn * hi)
        const int r1 = fast_div(row, p.rcp_bw), hi_ = fast_div(row, p.rcp_bwbn);
        const int wi = row - r1 * p.bw, ni = r1 - hi_ * p.bn;
        const int w = pw0 + wi, h = ph0 + hi_, n = pn0 + ni;
        const bool row_ok = w < p.W && h < p.H && n < p.N;
        const size_t row_off = (((size_t)n * p.H + h) * p.W + w) * p.ldc;
        bool ok = true;
        uint4 refq[MODE == MODE_DGRAD ? MaskRow<BN>::SLOTS : 1];
        const bool have_refq = prefetch_mask_row<MODE, BN>(p, row_ok, row_off, n0, n_hi, refq);
        if (lane == 0) ok = mbar_wait(acc_full, 0);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) {
            if (lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_EPI); }
        } else {
            SB_TLOG(threadIdx.x == 64, 4, clock64());      // accumulator complete
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
            // (the rings are idle once the accumulator is complete: their first bytes stage the output tile)
            store_row<MODE, BN>(p, taddr, row_ok, row_off, n0, n_hi, split, s_bias, p.tma_out ? smem : nullptr, row, have_refq ? refq : nullptr);
            if (p.tma_out) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
    }

    // ---- teardown: everyone meets here; TMEM is released on every path ----------------------------
    tc_fence_before();
    __syncthreads();
    if (p.tma_out && threadIdx.x == 64 && !*abort_flag) {
#pragma unroll
        for (int j = 0; j < BN / 64; ++j)
            if (n0 + 64 * j < n_hi) tma_store_4d(&mapC, smem0 + j * 16384, n0 + 64 * j, pw0, pn0, ph0);    // (c, w, n, h)
        tma_store_commit();
    }
    if (MODE == MODE_FWD && p.tma_out && p.pool_out != nullptr && warp >= 2 && !*abort_flag)
        pool_from_stage<BN>(p, smem, threadIdx.x - 64, n0, n_hi, pw0, ph0, pn0);     // reads the stage while the TMA stores read it too
    if (p.tma_out && threadIdx.x == 64 && !*abort_flag) tma_store_wait_read();
    SB_TLOG(threadIdx.x == 0, 5, clock64());   // epilogue done
    SB_TLOG(threadIdx.x == 0, 7, globaltimer_ns());
    SB_TRACE_END(2);
    if (*abort_flag) {
        // give copies that may still be in flight time to land before shared memory is released
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) { }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------
// The persistent halo kernel: one CTA walks many output tiles
// ------------------------------------------------------------------------------------------------
// A layer of many tiles (several per SM) spends, one tile per CTA, more time in per-CTA fixed work -- barrier and TMEM
// set-up (~1.3 us), the first operand round trip (~0.4 us), the accumulator drain and the epilogue (~1.5 us) -- than in
// a short main loop (1 - 3 us at 64 - 128 input channels).  Here a CTA is launched once per SM slot and walks the tiles
// t = blockIdx.x, blockIdx.x + gridDim.x, ... with
//   * the operand rings running on across tile boundaries (the producer warp starts the next tile's first groups while
//     the last ones of the current tile are still being multiplied), and
//   * two TMEM accumulators: the MMA warp fills accumulator (i & 1) for the i-th tile while the four epilogue warps
//     drain the other one (tcgen05.ld, bias + ReLU / mask, staging, TMA store, fused 2x2 pool), handing it back through
//     acc_empty[].
// The output tile is staged in its own shared-memory buffer (the rings are never idle here).  Unsplit reductions with
// the TMA-store epilogue only (the planner checks); everything else as in umma_halo_kernel, every wait bounded.
template <int BN> struct HaloPersistCfg {
    static constexpr int B_STAGE_BYTES = BN * 128;
    static constexpr int STAGE_OUT_BYTES = (BN / 64) * 16384;
    static constexpr int TMEM_COLS = 2 * BN;                 // 128, 256 or 512: powers of two
    static constexpr int smem_bytes(int a_stages, int a_slot_bytes, int b_stages)
    {
        return a_stages * a_slot_bytes + b_stages * B_STAGE_BYTES + STAGE_OUT_BYTES + 1024 /*alignment slack*/ + CTRL_BYTES;
    }
};

template <int MODE, int BN>
__global__ void __launch_bounds__(UMMA_THREADS, 1)
umma_halo_persist_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, const __grid_constant__ CUtensorMap mapC,
                         const UmmaParams p)
{
    static_assert(MODE == MODE_FWD || MODE == MODE_DGRAD, "halo kernel: forward and data gradient only");
    using C = HaloPersistCfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int SA = p.a_stages, SB = p.stages;
    const uint32_t row_step = (uint32_t)(p.bw * p.bn) * 128u;
    const uint32_t a_slot = (uint32_t)(p.bh + 2) * row_step;
    uint8_t* b_ring = smem + (size_t)SA * a_slot;
    uint8_t* stage_out = b_ring + (size_t)SB * C::B_STAGE_BYTES;
    uint8_t* ctrl = stage_out + C::STAGE_OUT_BYTES;
    uint64_t* b_full = (uint64_t*)ctrl;               // [MAX_STAGES]
    uint64_t* b_empty = b_full + MAX_STAGES;          // [MAX_STAGES]
    uint64_t* a_full = b_empty + MAX_STAGES;          // [MAX_A_STAGES]
    uint64_t* a_empty = a_full + MAX_A_STAGES;        // [MAX_A_STAGES]
    uint64_t* acc_full = a_empty + MAX_A_STAGES;      // [2]
    uint64_t* acc_empty = acc_full + 2;               // [2]
    uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    float* s_bias = (float*)(ctrl + 512);             // [BN]

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
#ifdef SB_CTA_TIMING
    unsigned long long* tlog = (p.timing != nullptr && blockIdx.x < 1024) ? p.timing + 16ull * blockIdx.x : nullptr;
#endif
    SB_TLOG(threadIdx.x == 0, 0, globaltimer_ns());
    SB_TRACE_BEGIN();
    SB_TLOG(threadIdx.x == 0, 6, clock64());
    const int m_tiles = p.tiles_w * p.tiles_h * p.tiles_n;
    const int n_tiles_total = m_tiles * p.tiles_per_shard;       // (tiles_per_shard = N tiles; conv layers have one shard)
    const int n_groups = p.total_chunks;                         // 3 * kchunks groups per tile
    const uint32_t smem0 = smem_u32(smem), bring0 = smem_u32(b_ring);

    // tile index -> pixel-box origin and first output column
    auto tile_coords = [&](int t, int& pw0, int& ph0, int& pn0, int& n0) {
        const int n_idx = fast_div_exact(t, p.rcp_mtiles, m_tiles);
        const int m_idx = t - n_idx * m_tiles;
        const int q1 = fast_div_exact(m_idx, p.rcp_tiles_w, p.tiles_w), q2 = fast_div_exact(m_idx, p.rcp_tiles_wh, p.tiles_w * p.tiles_h);
        pw0 = (m_idx - q1 * p.tiles_w) * p.bw;
        ph0 = (q1 - q2 * p.tiles_h) * p.bh;
        pn0 = q2 * p.bn;
        n0 = n_idx * BN;
    };

    // ---- one-time setup -----------------------------------------------------------------------
    if (warp == 0) {
        if (lane == 0) {
            for (int s = 0; s < SB; ++s) { mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 1); }
            for (int s = 0; s < SA; ++s) { mbar_init(&a_full[s], 1); mbar_init(&a_empty[s], 1); }
            for (int s = 0; s < 2; ++s) { mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], 1); }
            *abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, C::TMEM_COLS);
        tmem_relinquish();
    }
    pdl_wait();          // every thread that touches global memory waits for the predecessor kernel
    SB_TRACE_STAMP(trace_a);
    if (warp == 0) pdl_trigger();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    SB_TLOG(threadIdx.x == 0, 1, clock64());   // set-up done
    SB_TRACE_STAMP(trace_b);

    if (warp == 0) {
        // =========================== TMA producer ===============================================
        // (whole warp in lock-step, elected issue, one group per round: see umma_halo_kernel; the rings never reset)
        const uint32_t prod_el = elect_one() ? 1u : 0u;
        const uint32_t afull0 = smem_u32(&a_full[0]), bfull0 = smem_u32(&b_full[0]);
        int la_s = 0, lb_s = 0;
        uint32_t la_off = 0, lb_off = 0, pa_par = 1u, pb_par = 1u;
        bool ok = true;
        for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x) {
            int pw0, ph0, pn0, n0;
            tile_coords(t, pw0, ph0, pn0, n0);
            int kc = 0, dsi = 0;
            for (int g = 0; g < n_groups; ++g) {
                const int s1 = lb_s, s2 = s1 + 1 == SB ? 0 : s1 + 1, s3 = s2 + 1 == SB ? 0 : s2 + 1;
                const uint32_t p1 = pb_par, p2 = s2 == 0 ? p1 ^ 1u : p1, p3 = s3 == 0 ? p2 ^ 1u : p2;
                const bool w0 = mbar_try_wait(&a_empty[la_s], pa_par), w1 = mbar_try_wait(&b_empty[s1], p1),
                           w2 = mbar_try_wait(&b_empty[s2], p2), w3 = mbar_try_wait(&b_empty[s3], p3);
                if (!__all_sync(0xffffffffu, (w0 && w1 && w2 && w3) ? 1 : 0)) {
                    ok = __all_sync(0xffffffffu, (mbar_wait(&a_empty[la_s], pa_par) && mbar_wait(&b_empty[s1], p1) &&
                                                  mbar_wait(&b_empty[s2], p2) && mbar_wait(&b_empty[s3], p3)) ? 1 : 0) != 0;
                    if (!ok) break;
                }
                {
                    const uint32_t bar = afull0 + 8u * (uint32_t)la_s;
                    mbar_expect_tx_el(bar, a_slot, prod_el);
                    tma_load_4d_el(&mapA, smem0 + la_off, bar, kc * 64, pw0 + dsi - 1, pn0, ph0 - 1, prod_el);    // (c, w, n, h)
                    ++la_s; la_off += a_slot;
                    if (la_s == SA) { la_s = 0; la_off = 0; pa_par ^= 1u; }
                }
#pragma unroll
                for (int j = 0; j < 3; ++j) {
                    const int tap = MODE == MODE_FWD ? 3 * j + dsi : 3 * (2 - j) + (2 - dsi);
                    const uint32_t dst = bring0 + lb_off, bar = bfull0 + 8u * (uint32_t)lb_s;
                    mbar_expect_tx_el(bar, (uint32_t)C::B_STAGE_BYTES, prod_el);
                    if (MODE == MODE_FWD) {
                        tma_load_4d_el(&mapB, dst, bar, tap * p.w_cols + kc * 64, n0, 0, 0, prod_el);
                    } else {
#pragma unroll
                        for (int jj = 0; jj < BN / 64; ++jj)
                            tma_load_4d_el(&mapB, dst + jj * 8192, bar, tap * p.w_cols + n0 + 64 * jj, kc * 64, 0, 0, prod_el);
                    }
                    ++lb_s; lb_off += (uint32_t)C::B_STAGE_BYTES;
                    if (lb_s == SB) { lb_s = 0; lb_off = 0; pb_par ^= 1u; }
                }
                if (++dsi == 3) { dsi = 0; ++kc; }
            }
        }
        if (!ok && lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_TMA); }
        SB_TRACE_STAMP(trace_c);
        __syncwarp();
    } else if (warp == 1) {
        // =========================== MMA issuer =================================================
        constexpr uint32_t idesc = make_idesc(BN, 0, MODE != MODE_FWD);
        const uint32_t elected = elect_one() ? 1u : 0u;
        const uint64_t dA0 = make_desc(smem0, 16);
        const uint64_t dB0 = (MODE == MODE_FWD) ? make_desc(bring0, 16) : make_desc(bring0, 8192);
        const uint32_t a_hi = (uint32_t)(dA0 >> 32), b_hi = (uint32_t)(dB0 >> 32);
        const uint32_t a_lo0 = (uint32_t)dA0, b_lo0 = (uint32_t)dB0;
        constexpr uint32_t A_STEP = 32u >> 4, B_STEP = ((MODE == MODE_FWD) ? 32u : 2048u) >> 4;
        constexpr uint32_t BSTAGE16 = (uint32_t)C::B_STAGE_BYTES >> 4;
        const uint32_t aslot16 = a_slot >> 4, rowstep16 = row_step >> 4;
        int sa = 0, sb_ = 0;
        uint32_t pha = 0, phb = 0, aoff = 0, boff = 0;
        bool ok = true;
        int i = 0;                                  // tiles this CTA has started
        for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x, ++i) {
            const int buf = i & 1;
            // the epilogue must have drained this accumulator's previous tile (use u of a buffer waits for release u - 1;
            // a fresh barrier reports the phase before its first as complete)
            ok = __all_sync(0xffffffffu, mbar_wait(&acc_empty[buf], (uint32_t)(((i >> 1) + 1) & 1)) ? 1 : 0) != 0;
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
            for (int g = 0; g < n_groups; ++g) {
                const int s1 = sb_, s2 = s1 + 1 == SB ? 0 : s1 + 1, s3 = s2 + 1 == SB ? 0 : s2 + 1;
                const uint32_t p1 = phb, p2 = s2 == 0 ? p1 ^ 1u : p1, p3 = s3 == 0 ? p2 ^ 1u : p2;
                const uint32_t o1 = boff, o2 = s2 == 0 ? 0u : o1 + BSTAGE16, o3 = s3 == 0 ? 0u : o2 + BSTAGE16;
                const bool w0 = mbar_try_wait(&a_full[sa], pha), w1 = mbar_try_wait(&b_full[s1], p1), w2 = mbar_try_wait(&b_full[s2], p2),
                           w3 = mbar_try_wait(&b_full[s3], p3);
                if (!__all_sync(0xffffffffu, (w0 && w1) ? 1 : 0)) {
                    ok = __all_sync(0xffffffffu, (mbar_wait(&a_full[sa], pha) && mbar_wait(&b_full[s1], p1)) ? 1 : 0) != 0;
                    if (!ok) break;
                }
                tc_fence_after();
                const uint32_t alo = a_lo0 + aoff;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_bf16_lohi(d_tmem, alo + kk * A_STEP, a_hi, b_lo0 + o1 + kk * B_STEP, b_hi, idesc, (g > 0 || kk > 0) ? 1u : 0u, elected);
                if (elected) umma_commit(&b_empty[s1]);
                if (!__all_sync(0xffffffffu, w2 ? 1 : 0)) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&b_full[s2], p2) ? 1 : 0) != 0;
                    if (!ok) break;
                    tc_fence_after();
                }
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_bf16_lohi(d_tmem, alo + rowstep16 + kk * A_STEP, a_hi, b_lo0 + o2 + kk * B_STEP, b_hi, idesc, 1u, elected);
                if (elected) umma_commit(&b_empty[s2]);
                if (!__all_sync(0xffffffffu, w3 ? 1 : 0)) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&b_full[s3], p3) ? 1 : 0) != 0;
                    if (!ok) break;
                    tc_fence_after();
                }
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_bf16_lohi(d_tmem, alo + 2 * rowstep16 + kk * A_STEP, a_hi, b_lo0 + o3 + kk * B_STEP, b_hi, idesc, 1u, elected);
                if (elected) {
                    umma_commit(&b_empty[s3]);
                    umma_commit(&a_empty[sa]);
                }
                __syncwarp();
                sb_ = s3 + 1; boff = o3 + BSTAGE16; phb = p3;
                if (sb_ == SB) { sb_ = 0; boff = 0; phb ^= 1u; }
                ++sa; aoff += aslot16;
                if (sa == SA) { sa = 0; aoff = 0; pha ^= 1u; }
            }
            if (!ok) break;
            if (elected) umma_commit(&acc_full[buf]);   // this tile's accumulator is complete once the MMAs above have run
            __syncwarp();
        }
        if (!ok && lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_MMA); }
        __syncwarp();
    } else {
        // =========================== epilogue ===================================================
        const int q = warp % 4;               // TMEM lane quadrant of this warp
        const int row = q * 32 + lane;        // accumulator row handled by this thread
        const int t128 = threadIdx.x - 64;
        // tile row = wi + bw * (ni + bn * hi): the same for every tile
        const int r1 = fast_div(row, p.rcp_bw), hi_ = fast_div(row, p.rcp_bwbn);
        const int wi = row - r1 * p.bw, ni = r1 - hi_ * p.bn;
        bool ok = true;
        int i = 0;
        for (int t = blockIdx.x; t < n_tiles_total; t += gridDim.x, ++i) {
            const int buf = i & 1;
            int pw0, ph0, pn0, n0;
            tile_coords(t, pw0, ph0, pn0, n0);
            const int n_hi = p.n_total;
            const int w = pw0 + wi, h = ph0 + hi_, n = pn0 + ni;
            const bool row_ok = w < p.W && h < p.H && n < p.N;
            const size_t row_off = (((size_t)n * p.H + h) * p.W + w) * p.ldc;
            if (MODE == MODE_FWD && p.epi == UEPI_BIAS_ACT) {
                // (the previous tile's epilogue has passed its last barrier: nobody still reads the old bias values)
                for (int c = t128; c < BN; c += 128) s_bias[c] = (n0 + c < n_hi) ? p.bias[n0 + c] : 0.f;
            }
            uint4 refq[MODE == MODE_DGRAD ? MaskRow<BN>::SLOTS : 1];
            const bool have_refq = prefetch_mask_row<MODE, BN>(p, row_ok, row_off, n0, n_hi, refq);
            if (lane == 0) ok = mbar_wait(&acc_full[buf], (uint32_t)((i >> 1) & 1));
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) {
                if (lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_EPI); }
            }
            epi_bar_sync();                       // bias staged; a timeout seen by any epilogue warp is seen by all below
            if (*abort_flag) break;
            SB_TLOG(t128 == 0 && i < 4, 8 + 2 * i, clock64());      // accumulator of tile i complete
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN);
            store_row<MODE, BN>(p, taddr, row_ok, row_off, n0, n_hi, 0, s_bias, stage_out, row, have_refq ? refq : nullptr);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            tc_fence_before();
            epi_bar_sync();                       // the tile is staged and every warp has finished reading the accumulator
            if (t128 == 0) {
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&acc_empty[buf])) : "memory");   // accumulator free
#pragma unroll
                for (int j = 0; j < BN / 64; ++j)
                    if (n0 + 64 * j < n_hi) tma_store_4d(&mapC, smem_u32(stage_out) + j * 16384, n0 + 64 * j, pw0, pn0, ph0);    // (c, w, n, h)
                tma_store_commit();
            }
            if (MODE == MODE_FWD && p.pool_out != nullptr) pool_from_stage<BN>(p, stage_out, t128, n0, n_hi, pw0, ph0, pn0);
            if (t128 == 0) tma_store_wait_read();
            epi_bar_sync();                       // the stage may be overwritten by the next tile
            SB_TLOG(t128 == 0 && i < 4, 9 + 2 * i, clock64());      // epilogue of tile i done
        }
    }

    // ---- teardown: everyone meets here; TMEM is released on every path ----------------------------
    tc_fence_before();
    __syncthreads();
    SB_TLOG(threadIdx.x == 0, 5, clock64());
    SB_TLOG(threadIdx.x == 0, 7, globaltimer_ns());
    SB_TRACE_END(3);
    if (*abort_flag) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) { }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------
// The CTA-pair kernel (FWD / DGRAD): tcgen05.mma.cta_group::2
// ------------------------------------------------------------------------------------------------
// Two CTAs of a cluster -- neighbouring M tiles with the same N tile and split -- run as one 256 x BN MMA.
// Each CTA fetches its own 128-row A tile but only HALF of the B tile (BN/2 columns); the tensor core reads
// both halves across the pair, so the weight-side operand crosses L2 -> shared memory once per pair instead
// of once per CTA (the operand ring is bound by each SM's L2 read bandwidth).  Protocol:
//   * both producers aim their TMA completions at the LEADER's (cluster rank 0) full[s] barrier, which
//     expects the bytes of both CTAs;
//   * the leader's MMA thread issues cta_group::2 MMAs (D rows 0..127 land in the leader's TMEM, rows
//     128..255 in the peer's, same column range) and releases ring slot s in BOTH CTAs with a multicast commit;
//   * each CTA's epilogue warps read their own TMEM and write their own 128 output rows.
// No load uses multicast.  All waits are bounded as in the single-CTA kernel.
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t ld_cluster_u32(uint32_t caddr)
{
    uint32_t v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(caddr) : "memory");
    return v;
}
// TMA load whose completion may signal a barrier in the peer CTA (`bar_caddr` is a shared::cluster address)
__device__ __forceinline__ void tma_load_4d_pair(const CUtensorMap* map, void* dst, uint32_t bar_caddr, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(bar_caddr), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair_el(const CUtensorMap* map, uint32_t dst_saddr, uint32_t bar_caddr, int c0, int c1, int c2, int c3,
                                                    uint32_t elected)
{
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %7, 0;\n\t"
        "@q cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];\n\t}"
        ::"r"(dst_saddr), "l"(map), "r"(bar_caddr), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(elected)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrives (once the MMAs issued so far have completed) on the barrier at this offset in both CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar)
{
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(mask) : "memory");
}

template <int BN> struct PairCfg {
    static constexpr int B_HALF_BYTES = BN * 64;                       // BN/2 rows (or K x BN/2 columns) of 128 bytes
    static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_HALF_BYTES;
    static constexpr int MAX_STAGES_FIT = (BN >= 256) ? 6 : 8;
    static constexpr int TMEM_COLS = BN;
    static constexpr int smem_bytes(int stages) { return stages * STAGE_BYTES + 1024 + CTRL_BYTES; }
};

template <int MODE, int BN>
__global__ void __launch_bounds__(UMMA_THREADS, 1)
umma_pair_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, const __grid_constant__ CUtensorMap mapC,
                 const UmmaParams p)
{
    static_assert(BN == 128 || BN == 256, "pair kernel: N tiles of 128 or 256");
    using C = PairCfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int STAGES = p.stages;
    uint8_t* ctrl = smem + STAGES * C::STAGE_BYTES;
    uint64_t* full = (uint64_t*)ctrl;
    uint64_t* empty = full + MAX_STAGES;
    uint64_t* acc_full = empty + MAX_STAGES;
    uint32_t* tmem_slot = (uint32_t*)(acc_full + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    float* s_bias = (float*)(ctrl + 512);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t rank = cluster_ctarank();       // 0: leader (issues the MMAs), 1: peer
    const bool leader = rank == 0;

    // ---- tile coordinates (the pair shares blockIdx.y / blockIdx.z; its M tiles are 2j and 2j+1) ----
    // FWD / DGRAD: M tile = a 128-pixel box, N tile inside a shard.  WGRAD (conv layers, one tap per CTA, unsharded): M
    // tile = 128 gradient rows (output channels), N tile = BN input channels, blockIdx.z = tap * splits + split.
    const int m_idx = blockIdx.x, n_idx = blockIdx.y;
    int split = blockIdx.z, tap_fixed = 0, n0, n_hi, m0 = 0, m_hi = 0;
    if (MODE == MODE_WGRAD) {
        tap_fixed = blockIdx.z / p.splits;
        split = blockIdx.z % p.splits;
        n0 = n_idx * BN; n_hi = p.n_total;
        m0 = m_idx * 128; m_hi = p.m_total;
    } else {
        if (p.shards == 1) {
            n0 = n_idx * BN;
            n_hi = p.n_total;
        } else {
            const int sh = n_idx / p.tiles_per_shard, t = n_idx % p.tiles_per_shard;
            const int lo = (int)(((long)sh * p.n_total) / p.shards);
            n_hi = (int)(((long)(sh + 1) * p.n_total) / p.shards);
            n0 = lo + t * BN;
        }
    }
    if (n0 >= n_hi) return;   // uniform over the pair, before any barrier or TMEM allocation
    // an M index past the last tile (odd tile count) lands wholly out of bounds: zero loads, no stores
    const int mq1 = fast_div_exact(m_idx, p.rcp_tiles_w, p.tiles_w), mq2 = fast_div_exact(m_idx, p.rcp_tiles_wh, p.tiles_w * p.tiles_h);
    const int pw0 = (m_idx - mq1 * p.tiles_w) * p.bw;
    const int ph0 = (mq1 - mq2 * p.tiles_h) * p.bh;
    const int pn0 = mq2 * p.bn;
    const int k_begin = split * p.chunks_per_split;
    const int k_end = min(k_begin + p.chunks_per_split, p.total_chunks);
    const int n_iters = k_end - k_begin;

    // next load: FWD / DGRAD (k-chunk, tap); WGRAD pixel-box indices (w, h, n)
    int ld_a = 0, ld_b = 0, ld_c = 0;
    if (k_begin != 0) {
        if (MODE == MODE_WGRAD) {
            ld_a = k_begin % p.tiles_w; ld_b = (k_begin / p.tiles_w) % p.tiles_h; ld_c = k_begin / (p.tiles_w * p.tiles_h);
        } else {
            ld_a = k_begin % p.kchunks; ld_b = k_begin / p.kchunks;
        }
    }
    const int wg_dr = tap_fixed / 3 - 1, wg_ds = tap_fixed % 3 - 1;
    const int nb0 = n0 + (int)rank * (BN / 2);                     // first B column this CTA fetches
    const uint32_t full0_leader = map_to_cta(smem_u32(&full[0]), 0);
    // (whole producer warp in lock-step, elected issue: see the single-CTA kernel)
    int ld_s = 0;
    uint32_t ld_off = 0;
    const uint32_t smem0 = smem_u32(smem), full0 = smem_u32(&full[0]);
    auto issue_loads = [&](uint32_t el) {
        const uint32_t sa = smem0 + ld_off, sb = sa + A_STAGE_BYTES;
        const uint32_t bar = full0_leader + (uint32_t)ld_s * 8u;
        if (leader) mbar_expect_tx_el(full0 + 8u * (uint32_t)ld_s, 2u * (uint32_t)C::STAGE_BYTES, el);
        if (MODE == MODE_WGRAD) {
            // A = this CTA's 128 gradient rows of dy (two 64-channel boxes), B = its half of the shifted activations
            const int cw = ld_a * p.bw, ch = ld_b * p.bh, cn = ld_c * p.bn;
            tma_load_4d_pair_el(&mapA, sa, bar, m0, cw, ch, cn, el);
            tma_load_4d_pair_el(&mapA, sa + 8192, bar, m0 + 64, cw, ch, cn, el);
#pragma unroll
            for (int j = 0; j < BN / 128; ++j) tma_load_4d_pair_el(&mapB, sb + j * 8192, bar, nb0 + 64 * j, cw + wg_ds, ch + wg_dr, cn, el);
            if (++ld_a == p.tiles_w) { ld_a = 0; if (++ld_b == p.tiles_h) { ld_b = 0; ++ld_c; } }
        } else {
            const int kc = ld_a, tap = ld_b;
            int dr = 0, ds = 0;
            if (p.ntaps == 9) { const int r3 = tap >= 6 ? 2 : (tap >= 3 ? 1 : 0); dr = r3 - 1; ds = tap - 3 * r3 - 1; }
            if (MODE == MODE_DGRAD) { dr = -dr; ds = -ds; }
            tma_load_4d_pair_el(&mapA, sa, bar, kc * 64, pw0 + ds, ph0 + dr, pn0, el);
            if (MODE == MODE_FWD) {
                tma_load_4d_pair_el(&mapB, sb, bar, tap * p.w_cols + kc * 64, nb0, 0, 0, el);     // box of BN/2 rows
            } else {
#pragma unroll
                for (int j = 0; j < BN / 128; ++j) tma_load_4d_pair_el(&mapB, sb + j * 8192, bar, tap * p.w_cols + nb0 + 64 * j, kc * 64, 0, 0, el);
            }
            if (++ld_a == p.kchunks) { ld_a = 0; ++ld_b; }
        }
        ++ld_s; ld_off += (uint32_t)C::STAGE_BYTES;
        if (ld_s == STAGES) { ld_s = 0; ld_off = 0; }
    };
    const int preloaded = n_iters < STAGES ? n_iters : STAGES;

    // ---- one-time setup -----------------------------------------------------------------------
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(acc_full, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    cluster_sync_all();    // both CTAs' barriers exist before any copy or commit can signal them
    uint32_t prod_el = 0;
    if (warp == 0) {
        pdl_wait();
        pdl_trigger();
        prod_el = elect_one() ? 1u : 0u;
        for (int it = 0; it < preloaded; ++it) issue_loads(prod_el);
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, C::TMEM_COLS);
        tmem_relinquish_pair();
    }
    if (warp != 0) pdl_wait();
    if (MODE == MODE_FWD && p.epi == UEPI_BIAS_ACT && warp >= 2) {
        for (int c = threadIdx.x - 64; c < BN; c += 128) s_bias[c] = (n0 + c < n_hi) ? p.bias[n0 + c] : 0.f;
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();    // the peer's accumulator columns are allocated before the leader's first MMA writes them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // (two slots per round on rings of four or more stages: see the single-CTA kernel)
        int ws = 0;
        uint32_t wph = 0;
        const int batch = STAGES >= 4 ? 2 : 1;
        bool got = true;
        for (int it = preloaded; it < n_iters;) {
            const int nb = (batch == 2 && it + 1 < n_iters) ? 2 : 1;
            const int s2 = ws + 1 == STAGES ? 0 : ws + 1;
            const uint32_t p2 = s2 == 0 ? wph ^ 1u : wph;
            const bool w1 = mbar_try_wait(&empty[ws], wph), w2 = nb == 2 ? mbar_try_wait(&empty[s2], p2) : true;
            if (!__all_sync(0xffffffffu, (w1 && w2) ? 1 : 0)) {
                got = __all_sync(0xffffffffu, (mbar_wait(&empty[ws], wph) && (nb == 1 || mbar_wait(&empty[s2], p2))) ? 1 : 0) != 0;
                if (!got) break;
            }
            issue_loads(prod_el);
            if (nb == 2) issue_loads(prod_el);
            if (nb == 2) { ws = s2 + 1; wph = p2; } else { ws = ws + 1; }
            if (ws == STAGES) { ws = 0; wph ^= 1u; }
            it += nb;
        }
        if (!got && lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_TMA); }
        __syncwarp();
    } else if (warp == 1) {
        if (leader) {
            // (converged warp, elected issue: see the single-CTA kernel)
            constexpr uint32_t idesc = make_idesc(BN, MODE == MODE_WGRAD, MODE != MODE_FWD, 256);
            const uint32_t elected = elect_one() ? 1u : 0u;
            // the MMA addresses both accumulators with one TMEM address: the pair must have been given the same columns
            bool ok = ld_cluster_u32(map_to_cta(smem_u32(tmem_slot), 1)) == tmem_base;
            if (!ok && lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_PAIR_TMEM); }
            const uint32_t sa0 = smem_u32(smem);
            const uint64_t dA0 = (MODE == MODE_WGRAD) ? make_desc(sa0, 8192) : make_desc(sa0, 16);
            const uint64_t dB0 = (MODE == MODE_FWD) ? make_desc(sa0 + A_STAGE_BYTES, 16) : make_desc(sa0 + A_STAGE_BYTES, 8192);
            const uint32_t a_hi = (uint32_t)(dA0 >> 32), b_hi = (uint32_t)(dB0 >> 32);
            const uint32_t a_lo0 = (uint32_t)dA0, b_lo0 = (uint32_t)dB0;
            constexpr uint32_t A_STEP = ((MODE == MODE_WGRAD) ? 2048u : 32u) >> 4, B_STEP = ((MODE == MODE_FWD) ? 32u : 2048u) >> 4;
            constexpr uint32_t STAGE16 = (uint32_t)C::STAGE_BYTES >> 4;
            int s = 0;
            uint32_t ph = 0, off = 0;
            const int batch = STAGES >= 4 ? 2 : 1;
            const bool tmem_ok = ok;
            for (int it = 0; it < n_iters && ok;) {
                const int nb = (batch == 2 && it + 1 < n_iters) ? 2 : 1;
                const int s2 = s + 1 == STAGES ? 0 : s + 1;
                const uint32_t p2 = s2 == 0 ? ph ^ 1u : ph, off2 = s2 == 0 ? 0u : off + STAGE16;
                const bool w1 = mbar_try_wait(&full[s], ph), w2 = nb == 2 ? mbar_try_wait(&full[s2], p2) : true;
                if (!__all_sync(0xffffffffu, w1 ? 1 : 0)) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&full[s], ph) ? 1 : 0) != 0;
                    if (!ok) break;
                }
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_bf16_pair_lohi(tmem_base, a_lo0 + off + kk * A_STEP, a_hi, b_lo0 + off + kk * B_STEP, b_hi, idesc, (it > 0 || kk > 0) ? 1u : 0u, elected);
                if (elected) umma_commit_pair(&empty[s]);
                if (nb == 2) {
                    if (!__all_sync(0xffffffffu, w2 ? 1 : 0)) {
                        ok = __all_sync(0xffffffffu, mbar_wait(&full[s2], p2) ? 1 : 0) != 0;
                        if (!ok) break;
                        tc_fence_after();
                    }
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_bf16_pair_lohi(tmem_base, a_lo0 + off2 + kk * A_STEP, a_hi, b_lo0 + off2 + kk * B_STEP, b_hi, idesc, 1u, elected);
                    if (elected) umma_commit_pair(&empty[s2]);
                    s = s2; off = off2; ph = p2;
                }
                __syncwarp();
                ++s; off += STAGE16;
                if (s == STAGES) { s = 0; off = 0; ph ^= 1u; }
                it += nb;
            }
            if (tmem_ok && !ok && lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_MMA); }
            if (ok && elected) umma_commit_pair(acc_full);
            __syncwarp();
        }
    } else {
        const int q = warp % 4;
        const int row = q * 32 + lane;
        bool ok = true;
        // where this thread's accumulator row goes (computed while the main loop runs)
        bool row_ok;
        size_t row_off;
        if (MODE == MODE_WGRAD) {
            row_ok = (m0 + row) < m_hi;
            row_off = (size_t)split * p.split_stride + (size_t)(m0 + row) * p.ldc + (size_t)tap_fixed * p.w_cols;
        } else {
            const int r1 = fast_div(row, p.rcp_bw), ni = fast_div(row, p.rcp_bwbh);
            const int wi = row - r1 * p.bw, hi_ = r1 - ni * p.bh;
            const int w = pw0 + wi, h = ph0 + hi_, n = pn0 + ni;
            row_ok = w < p.W && h < p.H && n < p.N;
            row_off = (((size_t)n * p.H + h) * p.W + w) * p.ldc;
        }
        uint4 refq[MODE == MODE_DGRAD ? MaskRow<BN>::SLOTS : 1];
        const bool have_refq = prefetch_mask_row<MODE, BN>(p, row_ok, row_off, n0, n_hi, refq);
        if (lane == 0) ok = mbar_wait(acc_full, 0);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) {
            if (lane == 0) { *abort_flag = 1; atomicMax(p.status, (uint32_t)DEV_TIMEOUT_EPI); }
        } else {
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
            const bool staged_out = MODE != MODE_WGRAD && p.tma_out;
            store_row<MODE, BN>(p, taddr, row_ok, row_off, n0, n_hi, split, s_bias, staged_out ? smem : nullptr, row, have_refq ? refq : nullptr);
            if (staged_out) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
    }

    // ---- teardown ------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) { }
        __syncthreads();
    }
    cluster_sync_all();    // neither CTA leaves (or frees TMEM) while its partner may still signal or read it
    if (MODE != MODE_WGRAD && p.tma_out && threadIdx.x == 64 && !*abort_flag) {
#pragma unroll
        for (int j = 0; j < BN / 64; ++j)
            if (n0 + 64 * j < n_hi) tma_store_4d(&mapC, smem_u32(smem) + j * 16384, n0 + 64 * j, pw0, ph0, pn0);
        tma_store_commit();
    }
    if (MODE == MODE_FWD && p.tma_out && p.pool_out != nullptr && warp >= 2 && !*abort_flag)
        pool_from_stage<BN>(p, smem, threadIdx.x - 64, n0, n_hi, pw0, ph0, pn0);
    if (MODE != MODE_WGRAD && p.tma_out && threadIdx.x == 64 && !*abort_flag) tma_store_wait_read();   // shared memory may be released once the stores have read it; the writes complete with the grid
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------
// Host side: tensor maps and launch planning
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;
static char g_umma_err[256] = "";

static bool get_encode()
{
    if (g_encode) return true;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess) {
        snprintf(g_umma_err, sizeof(g_umma_err), "cuTensorMapEncodeTiled is not available from the driver");
        return false;
    }
    g_encode = (EncodeTiledFn)fn;
    return true;
}

// bf16 tensor with dims d[0..3] (innermost first, elements) and byte strides s[1..3]; box b[0..3].
static bool encode_map(CUtensorMap* map, const void* ptr, const uint64_t d[4], const uint64_t strides_bytes[3], const uint32_t box[4])
{
    if (!get_encode()) return false;
    cuuint64_t gd[4] = {d[0], d[1], d[2], d[3]};
    cuuint64_t gs[3] = {strides_bytes[0], strides_bytes[1], strides_bytes[2]};
    cuuint32_t bx[4] = {box[0], box[1], box[2], box[3]};
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), gd, gs, bx, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_umma_err, sizeof(g_umma_err), "cuTensorMapEncodeTiled failed (%d): dims %llu,%llu,%llu,%llu box %u,%u,%u,%u", (int)r,
                 (unsigned long long)d[0], (unsigned long long)d[1], (unsigned long long)d[2], (unsigned long long)d[3], box[0], box[1], box[2], box[3]);
        return false;
    }
    return true;
}
// Activation tensor [N][H][W][C] bf16 -> 4-D map (C, W, H, N) with a (64, bw, bh, bn) box.
static bool act_map(CUtensorMap* map, const void* ptr, int N, int H, int W, int C, int bw, int bh, int bn)
{
    uint64_t d[4] = {(uint64_t)C, (uint64_t)W, (uint64_t)H, (uint64_t)N};
    uint64_t s[3] = {(uint64_t)C * 2, (uint64_t)W * C * 2, (uint64_t)H * W * C * 2};
    uint32_t b[4] = {64, (uint32_t)bw, (uint32_t)bh, (uint32_t)bn};
    return encode_map(map, ptr, d, s, b);
}
// The same tensor with the dimensions listed as (C, W, N, H) and a (64, bw, bn, bh) box: the box then lies in shared
// memory as [h][n][w] rows, which is what the halo kernel wants (a shift in h is a whole number of bw * bn rows).
static bool act_map_hn(CUtensorMap* map, const void* ptr, int N, int H, int W, int C, int bw, int bh, int bn)
{
    uint64_t d[4] = {(uint64_t)C, (uint64_t)W, (uint64_t)N, (uint64_t)H};
    uint64_t s[3] = {(uint64_t)C * 2, (uint64_t)H * W * C * 2, (uint64_t)W * C * 2};
    uint32_t b[4] = {64, (uint32_t)bw, (uint32_t)bn, (uint32_t)bh};
    return encode_map(map, ptr, d, s, b);
}
// Row-major matrix [rows][cols] bf16 -> map (cols, rows, 1, 1) with a (64, box_rows, 1, 1) box.
static bool mat_map(CUtensorMap* map, const void* ptr, long rows, long cols, int box_rows)
{
    uint64_t d[4] = {(uint64_t)cols, (uint64_t)rows, 1, 1};
    uint64_t s[3] = {(uint64_t)cols * 2, (uint64_t)rows * cols * 2, (uint64_t)rows * cols * 2};
    uint32_t b[4] = {64, (uint32_t)box_rows, 1, 1};
    return encode_map(map, ptr, d, s, b);
}

// Row-major float matrix [rows][cols] -> map (cols, rows, 1, 1) with a (64, 128, 1, 1) box, no swizzle: 128 rows of 256 bytes.
static bool mat_map_f32(CUtensorMap* map, const void* ptr, long rows, long cols)
{
    if (!get_encode()) return false;
    cuuint64_t gd[4] = {(cuuint64_t)cols, (cuuint64_t)rows, 1, 1};
    cuuint64_t gs[3] = {(cuuint64_t)cols * 4, (cuuint64_t)rows * cols * 4, (cuuint64_t)rows * cols * 4};
    cuuint32_t bx[4] = {64, 128, 1, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<void*>(ptr), gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_umma_err, sizeof(g_umma_err), "cuTensorMapEncodeTiled (float matrix %ld x %ld) failed (%d)", rows, cols, (int)r);
        return false;
    }
    return true;
}

static int cdiv_i(long a, long b) { return (int)((a + b - 1) / b); }

// Pixel box (bw, bh, bn) with bw*bh*bn = target (a power of two): least padded volume, then widest rows.
static void choose_box(int W, int H, int N, int target, int* bw, int* bh, int* bn)
{
    double best = 1e300;
    int bbw = 1, bbh = 1;
    for (int w = 1; w <= target; w *= 2)
        for (int h = 1; w * h <= target; h *= 2) {
            int n = target / (w * h);
            double vol = (double)cdiv_i(W, w) * w * cdiv_i(H, h) * h * cdiv_i(N, n) * n;
            // prefer exact fits; among equal volumes prefer wider, then taller boxes (longer contiguous runs)
            double score = vol * (1.0 - 1e-6 * w - 1e-8 * h);
            if (score < best) { best = score; bbw = w; bbh = h; }
        }
    *bw = bbw; *bh = bbh; *bn = target / (bbw * bbh);
}

template <int MODE, int BN>
static cudaError_t launch_one(const UmmaOp& op, const UmmaParams& p, dim3 grid, cudaStream_t st)
{
    // (the attribute belongs to the device's copy of the function: set it once per device)
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(umma_kernel<MODE, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 MODE == MODE_WGRAD ? 227 * 1024 : Cfg<MODE, BN>::smem_bytes(Cfg<MODE, BN>::MAX_STAGES_FIT));
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    if (p.stages < 1 || p.stages > Cfg<MODE, BN>::MAX_STAGES_FIT) return cudaErrorInvalidValue;
    // (a weight gradient with the update folded in carries two parameter slab buffers behind its control block)
    const size_t smem = (size_t)Cfg<MODE, BN>::smem_bytes(p.stages) + (MODE == MODE_WGRAD && p.sgd_w != nullptr ? (size_t)UPD_EXTRA_SMEM : 0);
    if (smem > 227 * 1024) return cudaErrorInvalidValue;
    return pdl_launch(umma_kernel<MODE, BN>, grid, dim3(UMMA_THREADS), smem, st, op.mapA, op.mapB, op.mapC, op.mapD, p);
}

template <int MODE, int BN>
static cudaError_t launch_halo_one(const UmmaOp& op, const UmmaParams& p, dim3 grid, cudaStream_t st)
{
    const int a_slot = (p.bh + 2) * p.bw * p.bn * 128;
    const int smem = HaloCfg<BN>::smem_bytes(p.a_stages, a_slot, p.stages);
    if (p.a_stages < 1 || p.a_stages > MAX_A_STAGES || p.stages < 1 || p.stages > MAX_STAGES || smem > 227 * 1024) return cudaErrorInvalidValue;
    // (the attribute belongs to the device's copy of the function: set it once per device)
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(umma_halo_kernel<MODE, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    return pdl_launch(umma_halo_kernel<MODE, BN>, grid, dim3(UMMA_THREADS), (size_t)smem, st, op.mapA, op.mapB, op.mapC, p);
}
template <int MODE>
static cudaError_t launch_halo_mode(int bn, const UmmaOp& op, const UmmaParams& p, dim3 grid, cudaStream_t st)
{
    switch (bn) {
    case 64: return launch_halo_one<MODE, 64>(op, p, grid, st);
    case 128: return launch_halo_one<MODE, 128>(op, p, grid, st);
    case 256: return launch_halo_one<MODE, 256>(op, p, grid, st);
    default: return cudaErrorInvalidValue;
    }
}

template <int MODE, int BN>
static cudaError_t launch_halo_persist_one(const UmmaOp& op, const UmmaParams& p, dim3 grid, cudaStream_t st)
{
    const int a_slot = (p.bh + 2) * p.bw * p.bn * 128;
    const int smem = HaloPersistCfg<BN>::smem_bytes(p.a_stages, a_slot, p.stages);
    if (p.a_stages < 1 || p.a_stages > MAX_A_STAGES || p.stages < 3 || p.stages > MAX_STAGES || smem > 227 * 1024 || !p.tma_out || p.splits != 1)
        return cudaErrorInvalidValue;
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(umma_halo_persist_kernel<MODE, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    return pdl_launch(umma_halo_persist_kernel<MODE, BN>, grid, dim3(UMMA_THREADS), (size_t)smem, st, op.mapA, op.mapB, op.mapC, p);
}
template <int MODE>
static cudaError_t launch_halo_persist_mode(int bn, const UmmaOp& op, const UmmaParams& p, dim3 grid, cudaStream_t st)
{
    switch (bn) {
    case 64: return launch_halo_persist_one<MODE, 64>(op, p, grid, st);
    case 128: return launch_halo_persist_one<MODE, 128>(op, p, grid, st);
    case 256: return launch_halo_persist_one<MODE, 256>(op, p, grid, st);
    default: return cudaErrorInvalidValue;
    }
}

// CTA-pair launch: clusters of two CTAs along x, programmatic dependent launch as everywhere else.
template <int MODE, int BN>
static cudaError_t launch_pair_one(const UmmaOp& op, const UmmaParams& p, dim3 grid, cudaStream_t st)
{
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(umma_pair_kernel<MODE, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 PairCfg<BN>::smem_bytes(PairCfg<BN>::MAX_STAGES_FIT));
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    if (p.stages < 1 || p.stages > PairCfg<BN>::MAX_STAGES_FIT || (grid.x & 1u)) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(UMMA_THREADS);
    cfg.dynamicSmemBytes = (size_t)PairCfg<BN>::smem_bytes(p.stages);
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl_enabled() ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, umma_pair_kernel<MODE, BN>, op.mapA, op.mapB, op.mapC, p);
}
template <int MODE>
static cudaError_t launch_pair_mode(int bn, const UmmaOp& op, const UmmaParams& p, dim3 grid, cudaStream_t st)
{
    switch (bn) {
    case 128: return launch_pair_one<MODE, 128>(op, p, grid, st);
    case 256: return launch_pair_one<MODE, 256>(op, p, grid, st);
    default: return cudaErrorInvalidValue;
    }
}

template <int MODE>
static cudaError_t launch_mode(int bn, const UmmaOp& op, const UmmaParams& p, dim3 grid, cudaStream_t st)
{
    if (MODE == MODE_WGRAD && bn == 192) return launch_one<MODE_WGRAD, 192>(op, p, grid, st);
    switch (bn) {
    case 64: return launch_one<MODE, 64>(op, p, grid, st);
    case 128: return launch_one<MODE, 128>(op, p, grid, st);
    case 256: return launch_one<MODE, 256>(op, p, grid, st);
    default: return cudaErrorInvalidValue;
    }
}

// The op's full parameter block lives next to the tensor maps (host memory owned by the model).
struct OpBlock {
    UmmaParams p;
    int bn;
    int pair;      // FWD / DGRAD: run as CTA pairs (umma_pair_kernel); grid.x is then even
    int halo;      // 3x3 FWD / DGRAD: umma_halo_kernel (activation halos shared by the three taps of a filter column)
    int persist;   // ... its persistent variant: grid.x CTAs walk all tiles (umma_halo_persist_kernel)
    int upd_maps;  // FC WGRAD: mapC / mapD are float maps over the layer's master weights and momentum
    dim3 grid;
    long rows;     // output rows (pixels / batch rows) of a FWD / DGRAD op
};
static_assert(sizeof(OpBlock) <= sizeof(((UmmaOp*)nullptr)->blob), "UmmaOp::blob too small");
static OpBlock* blk(UmmaOp& op) { return (OpBlock*)op.blob; }
static const OpBlock* blk(const UmmaOp& op) { return (const OpBlock*)op.blob; }

#ifdef SB_CTA_TIMING
static unsigned long long* g_timing = nullptr;   // development builds only: set through umma_set_timing_buffer
static unsigned long long* g_trace = nullptr;
void umma_set_timing_buffer(void* dev_ptr) { g_timing = (unsigned long long*)dev_ptr; }
void umma_set_trace_buffer(void* dev_ptr) { g_trace = (unsigned long long*)dev_ptr; }
#endif

struct SgdFuse { float *w, *v; __nv_bfloat16* s; float lr, mu; };
static bool wgrad_sweep_ok(const OpBlock* b)
{
    const UmmaParams& pp = b->p;
    static const bool sweep_on = tune("SB_WGRAD_SWEEP", 1) != 0;
    const bool aligned = (pp.ldc & 3) == 0 && (pp.w_cols & 3) == 0 && (pp.n_total & 3) == 0 && (pp.split_stride & 3) == 0 &&
                         (((uintptr_t)pp.out) & 15) == 0;
    const long ring = (long)pp.stages * (A_STAGE_BYTES + b->bn * 128);
    return (sweep_on || pp.hn_order) && aligned && ring >= 32768;
}
static sb_status launch_op(const UmmaOp& op, cudaStream_t st, int64_t* launches = nullptr, const SgdFuse* fuse = nullptr)
{
    const OpBlock* b = blk(op);
    cudaError_t e;
    UmmaParams pp = b->p;
    if (fuse) {
        if (pp.mode != MODE_WGRAD || !b->upd_maps || b->pair || pp.splits != 1 || !pp.bias_fused || !wgrad_sweep_ok(b)) {
            snprintf(g_umma_err, sizeof(g_umma_err), "weight gradient with folded update asked for an op that cannot carry it");
            return SB_ERR_CUDA;
        }
        pp.sgd_w = fuse->w; pp.sgd_v = fuse->v; pp.sgd_s = fuse->s; pp.sgd_lr = fuse->lr; pp.sgd_mu = fuse->mu;
    }
    if (pp.mode == MODE_WGRAD && !b->pair) {
        pp.wg_sweep = wgrad_sweep_ok(b) ? 1 : 0;
        if (pp.hn_order && !pp.wg_sweep) {
            snprintf(g_umma_err, sizeof(g_umma_err), "filter-column weight gradient planned without the staged epilogue");
            return SB_ERR_CUDA;
        }
    }
#ifdef SB_CTA_TIMING
    pp.timing = g_timing;
    pp.trace = g_trace;
    {
        static const int only_mode = (int)tune("SB_TLOG_MODE", -1);      // log only kernels of one mode (0 fwd, 1 dgrad, 2 wgrad)
        if (only_mode >= 0 && pp.mode != only_mode) pp.timing = nullptr;
    }
    pp.dbg_skip = (int)tune("SB_HALO_SKIP", 0);
#endif
    if (pp.mode != MODE_WGRAD) {
        static const bool w_first_on = tune("SB_W_FIRST", 1) != 0;
        pp.w_first = (w_first_on && weights_first() && !b->pair && !b->persist) ? 1 : 0;
        pp.rcp_tiles_w = fast_rcp((uint32_t)pp.tiles_w);
        pp.rcp_tiles_wh = fast_rcp((uint32_t)(pp.tiles_w * pp.tiles_h));
        pp.rcp_bw = fast_rcp((uint32_t)pp.bw);
        pp.rcp_bwbh = fast_rcp((uint32_t)(pp.bw * pp.bh));
        pp.rcp_wb = fast_rcp((uint32_t)(pp.bw / 2));
        pp.rcp_wbhb = fast_rcp((uint32_t)((pp.bw / 2) * (pp.bh / 2)));
        pp.rcp_bwbn = fast_rcp((uint32_t)(pp.bw * pp.bn));
        pp.rcp_mtiles = fast_rcp((uint32_t)(pp.tiles_w * pp.tiles_h * pp.tiles_n));
    }
    if (b->halo && b->persist && b->p.mode == MODE_FWD) e = launch_halo_persist_mode<MODE_FWD>(b->bn, op, pp, b->grid, st);
    else if (b->halo && b->persist && b->p.mode == MODE_DGRAD) e = launch_halo_persist_mode<MODE_DGRAD>(b->bn, op, pp, b->grid, st);
    else if (b->halo && b->p.mode == MODE_FWD) e = launch_halo_mode<MODE_FWD>(b->bn, op, pp, b->grid, st);
    else if (b->halo && b->p.mode == MODE_DGRAD) e = launch_halo_mode<MODE_DGRAD>(b->bn, op, pp, b->grid, st);
    else if (b->pair && b->p.mode == MODE_FWD) e = launch_pair_mode<MODE_FWD>(b->bn, op, pp, b->grid, st);
    else if (b->pair && b->p.mode == MODE_DGRAD) e = launch_pair_mode<MODE_DGRAD>(b->bn, op, pp, b->grid, st);
    else if (b->pair && b->p.mode == MODE_WGRAD) e = launch_pair_mode<MODE_WGRAD>(b->bn, op, pp, b->grid, st);
    else if (b->p.mode == MODE_FWD) e = launch_mode<MODE_FWD>(b->bn, op, pp, b->grid, st);
    else if (b->p.mode == MODE_DGRAD) e = launch_mode<MODE_DGRAD>(b->bn, op, pp, b->grid, st);
    else e = launch_mode<MODE_WGRAD>(b->bn, op, pp, b->grid, st);
    if (e == cudaSuccess && b->p.mode != MODE_WGRAD && b->p.splits > 1) {
        // ordered sum of the split partial sums + the epilogue the tensor-core kernel skipped
        SplitKEpiArgs a{};
        a.part = b->p.part; a.split_stride = (size_t)b->p.split_stride; a.splits = b->p.splits;
        a.rows = b->rows; a.N = b->p.n_total;
        a.epi = b->p.epi == UEPI_BIAS_ACT ? EPI_BIAS_ACT : EPI_MASK;
        a.bias = b->p.bias; a.relu = b->p.relu; a.ref = b->p.ref; a.out = b->p.out; a.out_f32 = b->p.out_f32;
        e = launch_splitk_epilogue(a, st);
        if (launches) ++*launches;
    }
    if (e != cudaSuccess) {
        snprintf(g_umma_err, sizeof(g_umma_err), "tensor-core launch failed: %s", cudaGetErrorString(e));
        return SB_ERR_CUDA;
    }
    return SB_OK;
}

const char* umma_last_error() { return g_umma_err; }

// Self-test of the bounded-wait path: one CTA waits on an mbarrier that nothing will ever complete, with the same
// polling loop as the pipeline waits but a limit of `limit_ns`; when the limit passes it records DEV_TIMEOUT_EPI in the
// status word and returns normally, exactly as a stalled pipeline would.
__global__ void __launch_bounds__(32) wait_probe_kernel(uint32_t* status, unsigned long long limit_ns)
{
    __shared__ uint64_t never;
    if (threadIdx.x == 0) {
        mbar_init(&never, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const uint64_t t0 = globaltimer_ns();
        bool done = false;
        for (uint32_t it = 0; it < (1u << 28) && !done; ++it) {
            done = mbar_try_wait(&never, 0);
            if ((it & 255u) == 255u && globaltimer_ns() - t0 > limit_ns) break;
        }
        if (!done) atomicMax(status, (uint32_t)DEV_TIMEOUT_EPI);
    }
}
cudaError_t launch_wait_probe(uint32_t* status, unsigned long long limit_ns, cudaStream_t st)
{
    wait_probe_kernel<<<1, 32, 0, st>>>(status, limit_ns);
    return cudaGetLastError();
}

// Tile plan of a FWD / DGRAD GEMM: N tile, reduction split and ring depth.
//  * N tile as wide as the column count allows (operand traffic from L2 per FLOP falls with the tile width),
//  * if that leaves fewer CTAs than ~0.8 waves, split the reduction over blockIdx.z (float partial sums,
//    reduced in split order by splitk_epilogue) while every CTA keeps at least 4 k-iterations,
//  * ring depth = k-iterations per CTA, capped by what fits; for grids of several waves the ring is kept
//    shallow enough that two CTAs share an SM, so one CTA's epilogue overlaps the other's main loop.
struct TilePlan { int bn, splits, cps, stages, pair, halo, a_stages, persist, persist_ctas; };
// Backward kernels of the two concurrent streams share SMs only if two CTAs fit side by side (shared
// memory <= ~110 KB each, TMEM columns <= 256 each): SB_BWD_COHABIT=0 gives every kernel the full ring again.
static bool bwd_cohabit()
{
    static const bool on = tune("SB_BWD_COHABIT", 1) != 0;
    return on;
}
static int cohabit_stages(int bn) { return bn >= 192 ? 2 : (bn >= 128 ? 3 : 4); }

// Cost model behind the tile plan (micro-seconds), fitted to a sweep of N-tile width x split count over the
// VGG-16 / CIFAR layers (isolated launches, 5 us of event overhead removed):
//   * one k-iteration of a CTA that has an SM to itself costs 0.38 / 0.315 / 0.245 us for 256 / 128 / 64 columns
//     (operand bytes through the SM's L2 port; before the MMAs were issued from a converged warp it was ~0.45 us
//     whatever the width);
//   * two CTAs sharing an SM each run at ~1/1.6 of that rate;
//   * a CTA carries ~3 us of fixed work (start, first loads, drain, epilogue);
//   * a split reduction costs a second kernel (~4 us) plus ~0.5 us per MB of float partial sums written and read back
//     (8.4 MB -> 7 us, 16.8 MB -> 9 us, 33.5 MB -> 27 us measured).
static double plan_cost(int bn, int s, int n_cols_per_shard, int shards, long m_tiles, int k_iters)
{
    const long ctas = m_tiles * cdiv_i(n_cols_per_shard, bn) * shards * s;
    const double per_sm = (bn < 256 && ctas >= 296) ? 2.0 : 1.0;
    const double waves = (double)cdiv_i(ctas, (long)(148 * per_sm));
    const double t_iter = bn >= 256 ? 0.38 : (bn >= 128 ? 0.315 : 0.245);
    const double partial_mb = (double)s * (double)m_tiles * 128.0 * (double)n_cols_per_shard * shards * 4.0 / 1.0e6;
    const double mb_us = 0.5;
    return waves * (cdiv_i(k_iters, s) * t_iter * (per_sm > 1.0 ? 1.6 : 1.0) + 3.0) + (s > 1 ? 4.0 + mb_us * partial_mb : 0.0);
}
static TilePlan plan_tiles(int n_cols_per_shard, int shards, long m_tiles, int k_iters, bool backward, bool force_pair)
{
    TilePlan t;
    int best_bn = 64, best_s = 1;
    {
        double best = 1e300;
        for (int bn = 64; bn <= 256; bn *= 2) {
            if (bn > 64 && bn / 2 >= n_cols_per_shard) break;      // never wider than the columns need
            if (force_pair && bn < 256 && bn < n_cols_per_shard) continue;   // forced pairs: the widest tile only
            for (int s = 1; s <= 32 && (s == 1 || k_iters / s >= 4); s *= 2) {
                const double c = plan_cost(bn, s, n_cols_per_shard, shards, m_tiles, k_iters);
                if (c < best - 1e-9) { best = c; best_bn = bn; best_s = s; }
            }
        }
    }
    t.bn = best_bn;
    const long tiles = m_tiles * cdiv_i(n_cols_per_shard, t.bn) * shards;
    t.cps = cdiv_i(k_iters, best_s);
    t.splits = cdiv_i(k_iters, t.cps);
    const int fit = t.bn >= 256 ? 4 : (t.bn >= 128 ? 6 : 8);
    int st = t.cps < fit ? t.cps : fit;
    if (tiles * t.splits >= 296) {               // >= 2 waves: prefer two resident CTAs per SM
        const int two = t.bn >= 256 ? 2 : (t.bn >= 128 ? 3 : 4);
        if (t.bn < 256 && st > two) st = two;
    }
    static const bool fwd_too = tune("SB_FWD_COHABIT", 0) != 0;
    // (a grid that leaves SMs idle need not share its SMs: the other stream's CTAs find free ones; SB_COHABIT_MIN_CTAS)
    static const long cohabit_min = (long)tune("SB_COHABIT_MIN_CTAS", 100);
    if ((backward || fwd_too) && bwd_cohabit() && tiles * t.splits >= cohabit_min && st > cohabit_stages(t.bn)) st = cohabit_stages(t.bn);
    // Grids of more than one CTA per SM: measured, the co-residency of CTAs (their set-up, first loads and
    // epilogues overlap one another's main loops) is worth more than ring depth -- the 1024-CTA 64-wide layer runs
    // 28 us with 2 stages (4 CTAs per SM) against 37 us with 4 and 60 us with 8; beyond 3 stages no layer gains.
    // So the ring is cut down until the CTAs the grid asks for fit side by side (shared memory and TMEM columns
    // permitting), but never below a double buffer.  SB_STAGE_RULE=legacy keeps the older rule above.
    static const int min_stages = (int)tune("SB_MIN_STAGES", 2);
    {
        const long ctas = tiles * t.splits;
        long want = (ctas + 147) / 148;
        if (want > 512 / t.bn) want = 512 / t.bn;
        if (want > 8) want = 8;
        const int stage_bytes = 16384 + t.bn * 128;
        for (; want > 1; --want) {
            const int st_res = (int)((224 * 1024 / want - 3 * 1024) / stage_bytes);
            if (st_res >= min_stages) { if (st > st_res) st = st_res; break; }
        }
    }
    t.stages = st < 1 ? 1 : st;
    // CTA pairs: half the weight-side operand per CTA (a smaller stage, so a deeper ring).  Measured at VGG-16 /
    // ImageNet sizes the pair kernel is 1.2-1.3x faster where the N tile is 256 wide and the grid fills the
    // machine, slower for 128-wide tiles and for grids of less than a wave (two cluster barriers of fixed cost).
    // SB_PAIR=0 turns it off, SB_PAIR_MIN_CTAS moves the grid-size threshold.
    static const bool pair_on = tune("SB_PAIR", 1) != 0;
    static const long pair_min_ctas = (long)tune("SB_PAIR_MIN_CTAS", 1);
    t.pair = 0;
    t.halo = 0;
    t.a_stages = 0;
    t.persist = 0;
    t.persist_ctas = 0;
    // (SB_FLAG_FORCE_PAIR: every 128- or 256-wide tile, whatever the grid -- for tests at small sizes)
    if ((pair_on && t.bn == 256 && m_tiles % 2 == 0 && tiles * t.splits >= pair_min_ctas) || (force_pair && t.bn >= 128)) {
        t.pair = 1;
        const int pfit = t.bn >= 256 ? 6 : 8;
        int pst = t.cps < pfit ? t.cps : pfit;
        const int ptwo = t.bn >= 256 ? 3 : 4;      // two resident CTAs per SM
        if ((tiles * t.splits >= 296 || ((backward || fwd_too) && bwd_cohabit() && tiles * t.splits >= cohabit_min)) && pst > ptwo) pst = ptwo;
        t.stages = pst < 1 ? 1 : pst;
    }
    static const bool verbose = tune("SB_PLAN_VERBOSE", 0) != 0;
    if (verbose) fprintf(stderr, "plan: N/shard=%d shards=%d m_tiles=%ld k_iters=%d -> bn=%d splits=%d stages=%d pair=%d\n", n_cols_per_shard, shards, m_tiles, k_iters, t.bn, t.splits, t.stages, t.pair);
    return t;
}

// Pixel box of the halo kernel: bw * bh * bn = 128 (powers of two) with bw * bn a multiple of 8 (a shift by one image
// row is then a whole number of 8-row swizzle groups) and bh even (pooling windows inside the tile).  Least padded
// volume, weighted by the halo rows a box of that height fetches on top of its own ((bh + 2) / bh, of which the
// activations are about half of a CTA's operand bytes).
static bool choose_box_halo(int W, int H, int N, int* bw, int* bh, int* bn)
{
    double best = 1e300;
    bool found = false;
    for (int w = 1; w <= 128; w *= 2)
        for (int h = 2; w * h <= 128; h *= 2) {
            const int n = 128 / (w * h);
            if ((w * n) % 8 != 0 || n > 256 || w > 256) continue;
            const double vol = (double)cdiv_i(W, w) * w * cdiv_i(H, h) * h * cdiv_i(N, n) * n;
            const double score = vol * (1.0 + 1.0 / h) * (1.0 - 1e-6 * w);
            if (score < best) { best = score; *bw = w; *bh = h; *bn = n; found = true; }
        }
    return found;
}
// Tile plan of a halo-kernel op (see plan_tiles for the ideas): the reduction is 3 * kchunks groups of three taps.  The
// main loop is paced by the issuing warps, not by operand bytes: measured with the loads switched off it takes as long as
// with them, ~70 / 85 / 145 cycles per MMA for 64 / 128 / 256 columns (four MMAs per tap) once the producer and the
// MMA warp handle a whole group per round; the rings must then hold two groups of weight tiles or the producer, which
// waits for a whole group of free slots, falls behind (a ring of 4 runs at half the rate of a ring of 8).
static TilePlan plan_tiles_halo(int n_cols, long m_tiles, int kchunks, int a_slot_bytes, bool backward)
{
    TilePlan t{};
    t.halo = 1;
    const int groups = 3 * kchunks;
    double best = 1e300;
    int best_bn = 64, best_s = 1;
    static const double fixed_us = tune("SB_HALO_FIXED_US", 3.0), share_factor = tune("SB_HALO_SHARE", 1.6);
    static const double tap64 = tune("SB_HALO_TAP64", 0.16), tap128 = tune("SB_HALO_TAP128", 0.19), tap256 = tune("SB_HALO_TAP256", 0.33);
    for (int bn = 64; bn <= 256; bn *= 2) {
        if (bn > 64 && bn / 2 >= n_cols) break;
        const double t_tap = bn >= 256 ? tap256 : (bn >= 128 ? tap128 : tap64);
        for (int s = 1; s <= 32 && (s == 1 || groups / s >= 2); s *= 2) {
            const long ctas = m_tiles * cdiv_i(n_cols, bn) * s;
            const double per_sm = (bn < 256 && ctas >= 296) ? 2.0 : 1.0;
            const double waves = (double)cdiv_i(ctas, (long)(148 * per_sm));
            const double partial_mb = (double)s * (double)m_tiles * 128.0 * (double)n_cols * 4.0 / 1.0e6;
            const double c = waves * (cdiv_i(groups, s) * 3.0 * t_tap * (per_sm > 1.0 ? share_factor : 1.0) + fixed_us) + (s > 1 ? 4.0 + 0.5 * partial_mb : 0.0);
            if (c < best - 1e-9) { best = c; best_bn = bn; best_s = s; }
        }
    }
    {
        static const int f_bn = (int)tune("SB_HALO_BN", 0);
        if (f_bn > 0 && f_bn <= n_cols) { best_bn = f_bn; }
    }
    t.bn = best_bn;
    t.cps = cdiv_i(groups, best_s);            // groups per CTA
    t.splits = cdiv_i(groups, t.cps);
    const long ctas = m_tiles * cdiv_i(n_cols, t.bn) * t.splits;
    // Rings: as many CTAs side by side as the grid has per SM (TMEM columns and a two-group weight ring permitting, four
    // at most; backward grids of 100 CTAs or more leave room for a CTA of the weight-gradient streams), and within that
    // share of the shared memory the deepest rings.
    static const long cohabit_min = (long)tune("SB_COHABIT_MIN_CTAS", 100);
    long want = (ctas + 147) / 148;
    if (want > 512 / t.bn) want = 512 / t.bn;
    if (want > 4) want = 4;
    if (want < 2 && backward && bwd_cohabit() && ctas >= cohabit_min && t.bn < 256) want = 2;
    const int b_stage = t.bn * 128;
    int sa = 2, sb = 0;
    for (; want >= 1; --want) {
        const int budget = (int)(227 * 1024 / want) - 4 * 1024;
        sb = (budget - 2 * a_slot_bytes) / b_stage;
        if (sb >= 6 || want == 1) break;
    }
    if (sb > MAX_STAGES) sb = MAX_STAGES;
    if (sb < 3) sb = 3;
    if (want <= 1 && 227 * 1024 - 4 * 1024 - 3 * a_slot_bytes - sb * b_stage >= 0) sa = 3;
    {
        static const int f_sa = (int)tune("SB_HALO_SA", 0), f_sb = (int)tune("SB_HALO_SB", 0);
        if (f_sa > 0) sa = f_sa;
        if (f_sb > 0) sb = f_sb;
    }
    if (sa > t.cps) sa = t.cps;
    if (sb > 3 * t.cps) sb = 3 * t.cps;
    t.a_stages = sa;
    t.stages = sb;
    static const bool verbose = tune("SB_PLAN_VERBOSE", 0) != 0;
    if (verbose) fprintf(stderr, "plan: halo N=%d m_tiles=%ld kchunks=%d a_slot=%d -> bn=%d splits=%d a_stages=%d b_stages=%d (%.1f us)\n", n_cols, m_tiles, kchunks, a_slot_bytes, t.bn, t.splits, t.a_stages, t.stages, best);
    return t;
}

// Plan of the persistent halo kernel (layers of several tiles per SM, unsplit): 128-wide tiles where the layer has the
// columns (one CTA per SM with the deepest rings), 64-wide ones otherwise (two CTAs per SM with two-group rings).
static TilePlan plan_tiles_halo_persist(int n_cols, long m_tiles, int kchunks, int a_slot_bytes)
{
    TilePlan t{};
    t.halo = 1;
    t.persist = 1;
    static const int f_bn = (int)tune("SB_PERSIST_BN", 0);
    t.bn = f_bn > 0 ? f_bn : (n_cols >= 128 ? 128 : 64);
    t.splits = 1;
    t.cps = 3 * kchunks;
    const int b_stage = t.bn * 128, stage_out = (t.bn / 64) * 16384;
    int per_sm = 1, sa = 2, sb = 6;
    if (2 * (2 * a_slot_bytes + 6 * b_stage + stage_out + 4 * 1024) <= 227 * 1024 && 2 * 2 * t.bn <= 512) {
        per_sm = 2;
        sb = ((227 * 1024 / 2) - 4 * 1024 - stage_out - 2 * a_slot_bytes) / b_stage;
    } else {
        sa = 3;
        sb = (227 * 1024 - 4 * 1024 - stage_out - 3 * a_slot_bytes) / b_stage;
        if (sb < 6) { sa = 2; sb = (227 * 1024 - 4 * 1024 - stage_out - 2 * a_slot_bytes) / b_stage; }
    }
    if (sb > MAX_STAGES) sb = MAX_STAGES;
    if (sb < 3) sb = 3;
    {
        static const int f_sa = (int)tune("SB_PERSIST_SA", 0), f_sb = (int)tune("SB_PERSIST_SB", 0), f_per = (int)tune("SB_PERSIST_PER_SM", 0);
        if (f_sa > 0) sa = f_sa;
        if (f_sb > 0) sb = f_sb;
        if (f_per > 0) per_sm = f_per;
    }
    t.a_stages = sa;
    t.stages = sb;
    const long tiles = m_tiles * cdiv_i(n_cols, t.bn);
    const long slots = 148L * per_sm;
    t.persist_ctas = (int)(tiles < slots ? tiles : slots);
    static const bool verbose = tune("SB_PLAN_VERBOSE", 0) != 0;
    if (verbose) fprintf(stderr, "plan: halo persistent N=%d m_tiles=%ld kchunks=%d -> bn=%d a_stages=%d b_stages=%d ctas=%d (%ld tiles)\n", n_cols, m_tiles, kchunks, t.bn, t.a_stages, t.stages, t.persist_ctas, tiles);
    return t;
}

// Conv weight-gradient split count. Splitting the pixel (K) dimension fills more SMs but every split
// writes a float copy of the weight gradient and the ordered reduce reads them all back, so the choice is
// a small cost model: waves x (chunks per CTA x per-chunk operand time + fixed CTA cost) for the GEMM
// plus, when split, (S + 1) gradient copies through HBM/L2 and one more launch for the reduce.
// SB_WGRAD_SPLITS=legacy restores the older rule (fill 148 CTAs, at least 4 chunks per CTA).
static int wgrad_splits(long ctas_without_split, int total_chunks, int bn, size_t grad_floats, double* cost_out = nullptr)
{
    static const double reduce_gbs = tune("SB_WGRAD_REDUCE_GBS", 3000.0);
    static const double reduce_fixed = tune("SB_WGRAD_REDUCE_US", 3.0);
    static const double chunk_scale = tune("SB_WGRAD_CHUNK_SCALE", 1.0);
    const double chunk_us = chunk_scale * (16384.0 + bn * 128.0) / 122.0e3;     // bytes per chunk at ~122 GB/s of L2 per SM
    const double fixed_us = 3.0 + bn / 256.0 * 1.5;               // CTA start + drain + float epilogue
    double best = 1e30; int best_s = 1;
    for (int s = 1; s <= 256; ++s) {
        const int cps = cdiv_i(total_chunks, s);
        if (s > 1 && cps < 2) break;
        // Short kernels may take any split count (3 tap rows x 48 splits = 144 CTAs fill the machine: -1.2 % step at
        // CIFAR size); long ones (>= 256 chunks per CTA, ImageNet size) keep to powers of two, which leaves a third of
        // the SMs to the data-gradient kernel they run beside (filling the machine there measured +2.5 % step).
        if ((s & (s - 1)) != 0 && cps >= 256) continue;
        const int real_s = cdiv_i(total_chunks, cps);
        const long ctas = ctas_without_split * real_s;
        const long waves = (ctas + 147) / 148;
        // two resident CTAs share one SM's operand bandwidth: count a pair of waves as one at twice the chunk time
        double t = waves * (cps * chunk_us + fixed_us);
        if (real_s > 1) t += reduce_fixed + (real_s + 1) * (double)grad_floats * 4.0 / (reduce_gbs * 1e3);
        if (t < best) { best = t; best_s = real_s; }
    }
    static const bool verbose = tune("SB_PLAN_VERBOSE", 0) != 0;
    if (verbose) fprintf(stderr, "plan: wgrad base_ctas=%ld chunks=%d bn=%d grad=%zu -> splits=%d (%.1f us)\n", ctas_without_split, total_chunks, bn, grad_floats, best_s, best);
    if (cost_out) *cost_out = best;
    return best_s;
}

static bool conv_umma_ok(const ModelView& mv, const LayerView& lv, int layer)
{
    return mv.bf16 && !(mv.cfg->flags & SB_FLAG_FORCE_SIMT) && layer > 0 && lv.Cin % 64 == 0 && lv.Cout % 64 == 0;
}
static bool fc_umma_ok(const ModelView& mv, const LayerView& lv, int layer)
{
    // TMA needs 16-byte row strides: in and out multiples of 8; the reduce dims multiples of 64 keep every box row in bounds
    (void)layer;   // a first-layer FC reads the network input through a tensor map bound at forward time
    return mv.bf16 && !(mv.cfg->flags & SB_FLAG_FORCE_SIMT) && lv.in_f % 64 == 0 && lv.out_f % 8 == 0 && lv.out_f > 16;
}

// Geometry shared by the scratch sizing pass and the real planning pass.
struct ConvGeom {
    int bw, bh, bn, tw, th, tn;      // 128-pixel boxes (FWD / DGRAD M tiles)
    int halo;                        // the forward / data-gradient ops run on umma_halo_kernel (box chosen for it)
    long m_tiles;
    TilePlan fwd, dgrad;
    int cw, ch, cn, ctw, cth, ctn, total_chunks;   // 64-pixel boxes (WGRAD k-chunks)
    int wg_bn, wg_n_tiles, wg_m_tiles, wg_splits, wg_cps, wg_tap_group;
};
static ConvGeom conv_geom(const LayerView& lv, int B, bool force_pair, bool no_halo, bool force_persist)
{
    ConvGeom g;
    static const bool halo_on = tune("SB_HALO", 1) != 0;
    g.halo = 0;
    // The halo kernel wants deep rings (two groups of weight tiles in flight), so one CTA fills an SM's shared memory; a
    // grid of several CTAs per SM does better on the per-tap kernel, whose two-stage rings let four CTAs share an SM and
    // overlap their set-up and epilogue phases (measured at CIFAR size: 1024 tiles of 64 columns 25 us against 29 us).
    static const long halo_max_tiles = (long)tune("SB_HALO_MAX_TILES", 160);
    int hbw = 0, hbh = 0, hbn = 0;
    bool halo = halo_on && !force_pair && !no_halo && choose_box_halo(lv.W, lv.H, B, &hbw, &hbh, &hbn);
    static const bool persist_on = tune("SB_HALO_PERSIST", 1) != 0;
    static const long persist_max_width = (long)tune("SB_PERSIST_MAX_WIDTH", 128);
    bool persist = false;
    if (halo) {
        const long mt = (long)cdiv_i(lv.W, hbw) * cdiv_i(lv.H, hbh) * cdiv_i(B, hbn);
        const int widest = lv.Cout < lv.Cin ? lv.Cout : lv.Cin;
        const long tiles = mt * cdiv_i(widest, widest >= 128 ? 128 : 64);
        if (tiles > halo_max_tiles || force_persist) {
            // Four or more tiles per SM: the persistent variant (layers up to 128 channels wide; wider ones do better on the
            // per-tap kernel's CTA pairs with 256-column tiles).  Measured at CIFAR size, batch 128: the 1024-tile layer
            // 20.3 -> 16.3 us, the 256-tile layers 7.3 -> 9.0 and 12.8 -> 13.5 us (one or two tiles per CTA do not repay the
            // second accumulator's set-up); ImageNet-size step -3.6 %, batch 256 -2 %.
            static const long persist_min_tiles = (long)tune("SB_PERSIST_MIN_TILES", 4 * 148);
            persist = persist_on && (tiles >= persist_min_tiles || force_persist) && lv.Cout <= persist_max_width && lv.Cin <= persist_max_width &&
                      lv.Cout % 64 == 0 && lv.Cin % 64 == 0;
            if (!persist) halo = false;
        }
    }
    if (halo) {
        g.bw = hbw; g.bh = hbh; g.bn = hbn;
        g.halo = 1;
        g.tw = cdiv_i(lv.W, g.bw); g.th = cdiv_i(lv.H, g.bh); g.tn = cdiv_i(B, g.bn);
        g.m_tiles = (long)g.tw * g.th * g.tn;
        const int a_slot = (g.bh + 2) * g.bw * g.bn * 128;
        if (persist) {
            g.fwd = plan_tiles_halo_persist(lv.Cout, g.m_tiles, lv.Cin / 64, a_slot);
            g.dgrad = plan_tiles_halo_persist(lv.Cin, g.m_tiles, lv.Cout / 64, a_slot);
            if (force_persist) {      // (tests at small sizes: few CTAs, so that each walks several tiles and reuses both accumulators)
                if (g.fwd.persist_ctas > 3) g.fwd.persist_ctas = 3;
                if (g.dgrad.persist_ctas > 3) g.dgrad.persist_ctas = 3;
            }
        } else {
            g.fwd = plan_tiles_halo(lv.Cout, g.m_tiles, lv.Cin / 64, a_slot, false);
            g.dgrad = plan_tiles_halo(lv.Cin, g.m_tiles, lv.Cout / 64, a_slot, true);
        }
    } else {
        choose_box(lv.W, lv.H, B, 128, &g.bw, &g.bh, &g.bn);
        g.tw = cdiv_i(lv.W, g.bw); g.th = cdiv_i(lv.H, g.bh); g.tn = cdiv_i(B, g.bn);
        g.m_tiles = (long)g.tw * g.th * g.tn;
        g.fwd = plan_tiles(lv.Cout, 1, g.m_tiles, 9 * (lv.Cin / 64), false, force_pair);
        g.dgrad = plan_tiles(lv.Cin, 1, g.m_tiles, 9 * (lv.Cout / 64), true, force_pair);
    }
    choose_box(lv.W, lv.H, B, 64, &g.cw, &g.ch, &g.cn);
    g.ctw = cdiv_i(lv.W, g.cw); g.cth = cdiv_i(lv.H, g.ch); g.ctn = cdiv_i(B, g.cn);
    g.total_chunks = g.ctw * g.cth * g.ctn;
    g.wg_bn = lv.Cin >= 256 ? 256 : (lv.Cin >= 128 ? 128 : 64);
    g.wg_n_tiles = cdiv_i(lv.Cin, g.wg_bn);
    g.wg_m_tiles = cdiv_i(lv.Cout, 128);
    // 64 input channels: one CTA takes a whole filter row (three taps = 192 adjacent gradient columns), so the dy
    // tile is fetched once per three taps (SB_WGRAD_TAPS=1 restores one tap per CTA)
    static const bool taps1 = tune("SB_WGRAD_TAPS", 0) == 1;
    g.wg_tap_group = (lv.Cin == 64 && !taps1) ? 3 : 1;
    if (g.wg_tap_group == 3) g.wg_bn = 192;
    // 128 input channels and at most 128 output channels (one M tile, so no CTA pair): two adjacent taps per CTA as one
    // 256-column tile (dy fetched once per two taps; five tap groups, the last with tap 8 alone).  SB_WGRAD_TAPS=1 turns it off.
    // Taken for long reductions only (ImageNet-size layers: 613 -> 290 us alone); at CIFAR size the kernel alone is 15 %
    // faster but the step is not (its 96 KB ring and 256 TMEM columns leave the data-gradient kernel less room beside it).
    static const int taps2_min_chunks = (int)tune("SB_WGRAD_TAPS2_MIN_CHUNKS", 2048);
    if (lv.Cin == 128 && lv.Cout <= 128 && !taps1 && g.total_chunks >= taps2_min_chunks) { g.wg_tap_group = 2; g.wg_bn = 256; g.wg_n_tiles = 1; }
    const int tap_groups = (9 + g.wg_tap_group - 1) / g.wg_tap_group;
    double cost = 0.0;
    int s = wgrad_splits((long)g.wg_m_tiles * g.wg_n_tiles * tap_groups, g.total_chunks, g.wg_bn, (size_t)lv.n_w + lv.n_b, &cost);
    // a narrower N tile doubles the CTAs of a grid that leaves SMs idle (e.g. 512 channels at 4x4: 72 CTAs of 256
    // columns against 144 of 128): take it when the same model says it is faster (SB_WGRAD_NARROW=0 keeps the widest)
    // (reductions of 128 pixel chunks or more only: for the short ones -- 512 channels at 4x4 and 2x2, batch 128 / 256 -- the 72
    // wide CTAs leave half the SMs to the other streams, steps -0.6 %; the long ones of ImageNet-size inputs lose 1.3 % without it)
    static const bool narrow = tune("SB_WGRAD_NARROW", 1) != 0;
    static const int narrow_min_chunks = (int)tune("SB_WGRAD_NARROW_MIN_CHUNKS", 128);
    if (narrow && g.wg_tap_group == 1 && g.wg_bn == 256 && g.total_chunks >= narrow_min_chunks) {
        double cost2 = 0.0;
        const int n2 = cdiv_i(lv.Cin, 128);
        const int s2 = wgrad_splits((long)g.wg_m_tiles * n2 * 9, g.total_chunks, 128, (size_t)lv.n_w + lv.n_b, &cost2);
        if (cost2 < cost) { g.wg_bn = 128; g.wg_n_tiles = n2; s = s2; }
    }
    g.wg_cps = cdiv_i(g.total_chunks, s);
    g.wg_splits = cdiv_i(g.total_chunks, g.wg_cps);   // no empty trailing split
    return g;
}
struct FcGeom {
    int m_tiles;
    TilePlan fwd, dgrad;
};
static FcGeom fc_geom(const LayerView& lv, int B, int K, bool force_pair)
{
    FcGeom g;
    g.m_tiles = cdiv_i(B, 128);
    g.fwd = plan_tiles(cdiv_i(lv.out_f, K), K, g.m_tiles, lv.in_f / 64, false, force_pair);
    g.dgrad = plan_tiles(lv.in_f, 1, g.m_tiles, cdiv_i(lv.out_f, 64), true, force_pair);
    return g;
}

sb_status umma_plan_scratch(sb_model* m, size_t* floats)
{
    ModelView mv = model_view(m);
    size_t need = 0;
    auto upd = [&](size_t v) { if (v > need) need = v; };
    for (int i = 0; i < mv.n_layers; ++i) {
        LayerView lv = layer_view(m, i);
        if (lv.kind == SB_CONV3X3_RELU && conv_umma_ok(mv, lv, i)) {
            ConvGeom g = conv_geom(lv, mv.B, (mv.cfg->flags & SB_FLAG_FORCE_PAIR) != 0, (mv.cfg->flags & SB_FLAG_NO_HALO) != 0, (mv.cfg->flags & SB_FLAG_FORCE_PERSIST) != 0);
            const size_t pix = (size_t)mv.B * lv.H * lv.W;
            if (g.wg_splits > 1) upd((size_t)g.wg_splits * (lv.n_w + lv.n_b));
            if (g.fwd.splits > 1) upd((size_t)g.fwd.splits * pix * lv.Cout);
            if (g.dgrad.splits > 1) upd((size_t)g.dgrad.splits * pix * lv.Cin);
        } else if ((lv.kind == SB_FC_RELU || lv.kind == SB_FC) && fc_umma_ok(mv, lv, i)) {
            FcGeom g = fc_geom(lv, mv.B, lv.K, (mv.cfg->flags & SB_FLAG_FORCE_PAIR) != 0);
            if (g.fwd.splits > 1) upd((size_t)g.fwd.splits * mv.B * lv.out_f);
            if (g.dgrad.splits > 1) upd((size_t)g.dgrad.splits * mv.B * lv.in_f);
        }
    }
    *floats = need;
    return SB_OK;
}

static sb_status fail_plan() { return SB_ERR_CUDA; }

// Fills the split / ring fields of a FWD or DGRAD op from its tile plan.
static void apply_plan(OpBlock* b, const TilePlan& t, int k_iters, long m_tiles, int n_tiles_total, float* ws, size_t rows)
{
    // (the scratch for split partial sums was sized by umma_plan_scratch for the full batch; sub-batch plans are checked by the caller)
    UmmaParams& p = b->p;
    b->bn = t.bn;
    p.total_chunks = k_iters;
    p.chunks_per_split = t.cps;
    p.splits = t.splits;
    p.stages = t.stages;
    p.a_stages = t.a_stages;
    p.hn_order = t.halo;
    b->halo = t.halo;
    b->persist = t.persist;
    p.part = t.splits > 1 ? ws : nullptr;
    p.split_stride = (long)(rows * (size_t)p.n_total);
    b->pair = t.pair;
    b->grid = dim3((unsigned)(t.pair ? (m_tiles + 1) / 2 * 2 : m_tiles), (unsigned)n_tiles_total, (unsigned)t.splits);
    if (t.persist) b->grid = dim3((unsigned)t.persist_ctas, 1, 1);
    b->rows = (long)rows;
}

// TMA-store epilogue of a FWD / DGRAD op: possible when the output is bf16, the reduction is not split, every N tile
// ends on a 64-column slab boundary inside its shard, and the idle operand ring can hold the staged tile.
// SB_TMA_OUT=0 keeps the direct row stores.
static bool tma_out_ok(const OpBlock* b, int cols_per_shard, int shards)
{
    static const bool off = tune("SB_TMA_OUT", 1) == 0;
    const UmmaParams& p = b->p;
    if (off || p.out_f32 || p.splits > 1 || p.epi == UEPI_F32) return false;
    if (p.n_total % 64 != 0 || p.ldc % 64 != 0) return false;
    if (shards > 1 && (cols_per_shard % b->bn != 0 || p.n_total % shards != 0)) return false;
    if (b->halo && b->persist) return true;
    if (b->halo) return (long)p.a_stages * (p.bh + 2) * p.bw * p.bn * 128 + (long)p.stages * b->bn * 128 >= (long)(b->bn / 64) * 16384;
    const long stage_bytes = b->pair ? 16384 + b->bn * 64 : 16384 + b->bn * 128;
    return (long)p.stages * stage_bytes >= (long)(b->bn / 64) * 16384;
}

sb_status umma_plan_layers(sb_model* m, int first_layer)
{
    ModelView mv = model_view(m);
    if (!mv.bf16 || (mv.cfg->flags & SB_FLAG_FORCE_SIMT)) return SB_OK;
    const int B = mv.B;
    for (int i = first_layer; i < mv.n_layers; ++i) {
        LayerView lv = layer_view(m, i);
        UmmaLayer& um = *lv.um;
        const bool want_in_grad = i > 0;
        if (lv.kind == SB_CONV3X3_RELU && !conv_umma_ok(mv, lv, i) && conv_in_umma_supported(lv.Cin, lv.Cout)) {
            // input layer: the weight-gradient kernel fetches dy as [pixels][64] rows, 64 pixels per box
            static const bool off = tune("SB_CONV_IN_UMMA", 1) == 0;
            if (!off) {
                if (!mat_map(&um.wgrad.mapA, lv.dact, (long)B * lv.H * lv.W, lv.Cout, 64)) return fail_plan();
                if (!mat_map(&um.fwd.mapA, lv.act, (long)B * lv.H * lv.W, lv.Cout, 128)) return fail_plan();
                um.conv_in = true;
            }
        }
        if (lv.kind == SB_CONV3X3_RELU && conv_umma_ok(mv, lv, i)) {
            const ConvGeom g = conv_geom(lv, B, (mv.cfg->flags & SB_FLAG_FORCE_PAIR) != 0, (mv.cfg->flags & SB_FLAG_NO_HALO) != 0, (mv.cfg->flags & SB_FLAG_FORCE_PERSIST) != 0);
            const size_t pix = (size_t)B * lv.H * lv.W;
            // ---- forward ----
            {
                OpBlock* b = blk(um.fwd);
                memset(b, 0, sizeof(*b));
                UmmaParams& p = b->p;
                p.mode = MODE_FWD; p.ntaps = 9; p.bw = g.bw; p.bh = g.bh; p.bn = g.bn; p.W = lv.W; p.H = lv.H; p.N = B;
                p.tiles_w = g.tw; p.tiles_h = g.th; p.tiles_n = g.tn; p.kchunks = lv.Cin / 64; p.w_cols = lv.Cin;
                p.n_total = lv.Cout; p.shards = 1;
                p.tiles_per_shard = cdiv_i(lv.Cout, g.fwd.bn);
                p.epi = UEPI_BIAS_ACT; p.relu = 1; p.out_f32 = 0; p.out = lv.act; p.ldc = lv.Cout; p.bias = mv.Wm + lv.p_b;
                p.status = mv.status;
                apply_plan(b, g.fwd, g.halo ? 3 * p.kchunks : 9 * p.kchunks, g.m_tiles, p.tiles_per_shard, mv.ws, pix);
                if (g.halo) {
                    if (!act_map_hn(&um.fwd.mapA, lv.in_act, B, lv.H, lv.W, lv.Cin, g.bw, g.bh + 2, g.bn)) return fail_plan();
                } else if (!act_map(&um.fwd.mapA, lv.in_act, B, lv.H, lv.W, lv.Cin, g.bw, g.bh, g.bn)) return fail_plan();
                if (!mat_map(&um.fwd.mapB, mv.Sm + lv.p_w, lv.Cout, 9L * lv.Cin, b->pair ? b->bn / 2 : b->bn)) return fail_plan();
                if (tma_out_ok(b, lv.Cout, 1)) {
                    if (g.halo) {
                        if (!act_map_hn(&um.fwd.mapC, lv.act, B, lv.H, lv.W, lv.Cout, g.bw, g.bh, g.bn)) return fail_plan();
                    } else if (!act_map(&um.fwd.mapC, lv.act, B, lv.H, lv.W, lv.Cout, g.bw, g.bh, g.bn)) return fail_plan();
                    p.tma_out = 1;
                    // a 2x2 max-pool right above: pooled from the staged tile in the same kernel (SB_POOL_FUSE=0: separate kernel)
                    static const bool pool_fuse = tune("SB_POOL_FUSE", 1) != 0;
                    um.pool_fused = false;
                    if (pool_fuse && i + 1 < mv.n_layers && g.bw % 2 == 0 && g.bh % 2 == 0 && lv.W % 2 == 0 && lv.H % 2 == 0 && lv.Cout % 8 == 0) {
                        LayerView nx = layer_view(m, i + 1);
                        if (nx.kind == SB_MAXPOOL2 && nx.pool_idx != nullptr) {
                            p.pool_out = (__nv_bfloat16*)nx.act;
                            p.pool_idx = nx.pool_idx;
                            um.pool_fused = true;
                        }
                    }
                }
                um.fwd.enabled = true;
            }
            // ---- data gradient ----
            if (want_in_grad) {
                OpBlock* b = blk(um.dgrad);
                memset(b, 0, sizeof(*b));
                UmmaParams& p = b->p;
                p.mode = MODE_DGRAD; p.ntaps = 9; p.bw = g.bw; p.bh = g.bh; p.bn = g.bn; p.W = lv.W; p.H = lv.H; p.N = B;
                p.tiles_w = g.tw; p.tiles_h = g.th; p.tiles_n = g.tn; p.kchunks = lv.Cout / 64; p.w_cols = lv.Cin;
                p.n_total = lv.Cin; p.shards = 1;
                p.tiles_per_shard = cdiv_i(lv.Cin, g.dgrad.bn);
                p.epi = UEPI_MASK; p.out = lv.d_below; p.ldc = lv.Cin;
                p.ref = lv.below_relu ? (const __nv_bfloat16*)lv.in_act : nullptr;
                p.status = mv.status;
                apply_plan(b, g.dgrad, g.halo ? 3 * p.kchunks : 9 * p.kchunks, g.m_tiles, p.tiles_per_shard, mv.ws, pix);
                if (g.halo) {
                    if (!act_map_hn(&um.dgrad.mapA, lv.dact, B, lv.H, lv.W, lv.Cout, g.bw, g.bh + 2, g.bn)) return fail_plan();
                } else if (!act_map(&um.dgrad.mapA, lv.dact, B, lv.H, lv.W, lv.Cout, g.bw, g.bh, g.bn)) return fail_plan();
                if (!mat_map(&um.dgrad.mapB, mv.Sm + lv.p_w, lv.Cout, 9L * lv.Cin, 64)) return fail_plan();
                if (tma_out_ok(b, lv.Cin, 1)) {
                    if (g.halo) {
                        if (!act_map_hn(&um.dgrad.mapC, lv.d_below, B, lv.H, lv.W, lv.Cin, g.bw, g.bh, g.bn)) return fail_plan();
                    } else if (!act_map(&um.dgrad.mapC, lv.d_below, B, lv.H, lv.W, lv.Cin, g.bw, g.bh, g.bn)) return fail_plan();
                    p.tma_out = 1;
                }
                um.dgrad.enabled = true;
            }
            // ---- weight gradient ----
            {
                OpBlock* b = blk(um.wgrad);
                memset(b, 0, sizeof(*b));
                UmmaParams& p = b->p;
                p.mode = MODE_WGRAD; p.ntaps = 9; p.bw = g.cw; p.bh = g.ch; p.bn = g.cn; p.W = lv.W; p.H = lv.H; p.N = B;
                p.tiles_w = g.ctw; p.tiles_h = g.cth; p.tiles_n = g.ctn;
                p.total_chunks = g.total_chunks;
                p.w_cols = lv.Cin; p.n_total = lv.Cin * g.wg_tap_group; p.shards = 1; p.tiles_per_shard = 1;
                p.m_total = lv.Cout; p.m_shards = 1; p.m_tiles_per_shard = g.wg_m_tiles;
                p.tap_group = g.wg_tap_group;
                b->bn = g.wg_bn;
                p.splits = g.wg_splits;
                p.chunks_per_split = g.wg_cps;
                {
                    const int fit = b->bn >= 256 ? 4 : (b->bn >= 192 ? 5 : (b->bn >= 128 ? 6 : 8));
                    p.stages = g.wg_cps < fit ? g.wg_cps : fit;
                }
                {
                    // grids of fewer than ~100 CTAs leave the other streams whole SMs: no need to keep the ring shallow (measured: -1.5 % step)
                    static const long wg_cohabit_min = (long)tune("SB_WG_COHABIT_MIN_CTAS", 100);
                    const long ctas = (long)p.m_tiles_per_shard * g.wg_n_tiles * ((9 + p.tap_group - 1) / p.tap_group) * p.splits;
                    // (the filter-row kernel keeps its whole five-stage ring: with two slots per round the deeper ring is worth more
                    // than a neighbour on the SM -- steps -0.2 to -1.6 % against a ring cut to two or three 40 KB stages)
                    const int cap = b->bn == 192 ? 5 : cohabit_stages(b->bn);
                    if (bwd_cohabit() && ctas >= wg_cohabit_min && p.stages > cap) p.stages = cap;
                }
                p.epi = UEPI_F32; p.ldc = 9L * lv.Cin;
                // the bias gradient rides along: in the parameter arena the bias vector directly follows the
                // weights (Cout*9*Cin is a multiple of 64 here), and a split buffer uses the same layout
                p.split_stride = (long)(lv.n_w + lv.n_b);
                p.bias_fused = 1; p.bias_off = (long)lv.n_w;
                {
                    // CTA pairs over two neighbouring blocks of 128 output channels: each CTA fetches half of the
                    // activation tile (a smaller stage, a deeper ring in the same shared memory).  The pair kernel
                    // does not sum dy on the side, so the bias gradient is taken by a column-sum kernel (wgrad_pair).
                    static const bool wg_pair = tune("SB_WG_PAIR", 1) != 0;
                    // (long reductions only: below ~160 pixel chunks the pair's two cluster barriers and the separate column-sum
                    // kernel cost more than the halved activation fetch saves: CIFAR shape at batch 128 -1.4 % step with pairs,
                    // batch 256 +0.4 %, ImageNet shape +1.9 %)
                    static const int wg_pair_min_chunks = (int)tune("SB_WG_PAIR_MIN_CHUNKS", 160);
                    if (wg_pair && (g.total_chunks >= wg_pair_min_chunks || (mv.cfg->flags & SB_FLAG_FORCE_PAIR)) && p.tap_group == 1 && (b->bn == 128 || b->bn == 256) && g.wg_m_tiles % 2 == 0 && lv.Cout % 128 == 0) {
                        b->pair = 1;
                        p.bias_fused = 0;
                        const int pfit = b->bn >= 256 ? 6 : 8, ptwo = b->bn >= 256 ? 3 : 4;
                        int pst = g.wg_cps < pfit ? g.wg_cps : pfit;
                        const long ctas = (long)g.wg_m_tiles * g.wg_n_tiles * 9 * p.splits;
                        if (bwd_cohabit() && ctas >= 100 && pst > ptwo) pst = ptwo;
                        p.stages = pst < 1 ? 1 : pst;
                    }
                }
                p.out = p.splits > 1 ? (void*)mv.ws_wk[mv.n_wstreams > 0 ? i % mv.n_wstreams : 0] : (void*)(mv.Gm + lv.p_w);
                p.status = mv.status;
                b->grid = dim3((unsigned)p.m_tiles_per_shard, (unsigned)g.wg_n_tiles, (unsigned)((9 + p.tap_group - 1) / p.tap_group * p.splits));
                if ((size_t)p.splits * (lv.n_w + lv.n_b) > mv.ws_floats && p.splits > 1) return SB_ERR_ARENA_TOO_SMALL;
                // 64 input channels: one filter COLUMN per CTA instead of one filter row -- the three taps then share one
                // activation box with a halo row above and below (the three N panels of the MMA are windows into it) instead
                // of three boxes shifted in w.  Needs whole 8-row swizzle groups per image row of the box and the sweep epilogue.
                static const bool col_on = tune("SB_WG_COLUMN", 1) != 0;
                if (col_on && p.tap_group == 3 && !b->pair && (g.cw * g.cn) % 8 == 0 && (p.split_stride & 3) == 0 && (((uintptr_t)p.out) & 15) == 0 &&
                    !(mv.cfg->flags & SB_FLAG_NO_HALO)) {
                    p.hn_order = 1;
                    if (!act_map_hn(&um.wgrad.mapA, lv.dact, B, lv.H, lv.W, lv.Cout, g.cw, g.ch, g.cn)) return fail_plan();
                    if (!act_map_hn(&um.wgrad.mapB, lv.in_act, B, lv.H, lv.W, lv.Cin, g.cw, g.ch + 2, g.cn)) return fail_plan();
                } else {
                    if (!act_map(&um.wgrad.mapA, lv.dact, B, lv.H, lv.W, lv.Cout, g.cw, g.ch, g.cn)) return fail_plan();
                    if (!act_map(&um.wgrad.mapB, lv.in_act, B, lv.H, lv.W, lv.Cin, g.cw, g.ch, g.cn)) return fail_plan();
                }
                um.wgrad.enabled = true;
            }
        } else if ((lv.kind == SB_FC_RELU || lv.kind == SB_FC) && fc_umma_ok(mv, lv, i)) {
            const int K = lv.K;
            const FcGeom g = fc_geom(lv, B, K, (mv.cfg->flags & SB_FLAG_FORCE_PAIR) != 0);
            const int m_tiles = g.m_tiles;
            if (i == 0) lv.in_act = mv.stage_x;   // placeholder; rebound to the caller's input by umma_bind_input
            const bool fc_in_grad = i > 0 || (mv.cfg->flags & SB_FLAG_INPUT_GRAD);
            // ---- forward: Y[:, shard j] = X W_j^T + b_j ; N tiles enumerated per shard ----
            {
                OpBlock* b = blk(um.fwd);
                memset(b, 0, sizeof(*b));
                UmmaParams& p = b->p;
                p.mode = MODE_FWD; p.ntaps = 1; p.bw = 1; p.bh = 1; p.bn = 128; p.W = 1; p.H = 1; p.N = B;
                p.tiles_w = 1; p.tiles_h = 1; p.tiles_n = m_tiles; p.kchunks = lv.in_f / 64; p.w_cols = lv.in_f;
                p.n_total = lv.out_f; p.shards = K;
                p.tiles_per_shard = cdiv_i(cdiv_i(lv.out_f, K), g.fwd.bn);
                p.epi = UEPI_BIAS_ACT; p.relu = lv.relu ? 1 : 0; p.out_f32 = lv.kind == SB_FC; p.out = lv.act; p.ldc = lv.out_f;
                p.bias = mv.Wm + lv.p_b; p.status = mv.status;
                apply_plan(b, g.fwd, p.kchunks, m_tiles, p.tiles_per_shard * K, mv.ws, (size_t)B);
                if (p.splits > 1 && (size_t)p.splits * (size_t)p.split_stride > mv.ws_floats) return SB_ERR_ARENA_TOO_SMALL;
                if (!act_map(&um.fwd.mapA, lv.in_act, B, 1, 1, lv.in_f, 1, 1, 128)) return fail_plan();
                if (!mat_map(&um.fwd.mapB, mv.Sm + lv.p_w, lv.out_f, lv.in_f, b->pair ? b->bn / 2 : b->bn)) return fail_plan();
                if (tma_out_ok(b, cdiv_i(lv.out_f, K), K)) {
                    if (!act_map(&um.fwd.mapC, lv.act, B, 1, 1, lv.out_f, 1, 1, 128)) return fail_plan();
                    p.tma_out = 1;
                }
                um.fwd.enabled = true;
            }
            // ---- data gradient: dX = sum_j dY_j W_j = one reduction over the concatenated width ----
            if (fc_in_grad && lv.out_f % 8 == 0) {
                OpBlock* b = blk(um.dgrad);
                memset(b, 0, sizeof(*b));
                UmmaParams& p = b->p;
                p.mode = MODE_DGRAD; p.ntaps = 1; p.bw = 1; p.bh = 1; p.bn = 128; p.W = 1; p.H = 1; p.N = B;
                p.tiles_w = 1; p.tiles_h = 1; p.tiles_n = m_tiles; p.kchunks = cdiv_i(lv.out_f, 64); p.w_cols = lv.in_f;
                p.n_total = lv.in_f; p.shards = 1;
                p.tiles_per_shard = cdiv_i(lv.in_f, g.dgrad.bn);
                p.epi = UEPI_MASK; p.out = lv.d_below; p.ldc = lv.in_f;
                p.ref = lv.below_relu ? (const __nv_bfloat16*)lv.in_act : nullptr;
                p.status = mv.status;
                apply_plan(b, g.dgrad, p.kchunks, m_tiles, p.tiles_per_shard, mv.ws, (size_t)B);
                if (p.splits > 1 && (size_t)p.splits * (size_t)p.split_stride > mv.ws_floats) return SB_ERR_ARENA_TOO_SMALL;
                if (!act_map(&um.dgrad.mapA, lv.dact, B, 1, 1, lv.out_f, 1, 1, 128)) return fail_plan();
                if (!mat_map(&um.dgrad.mapB, mv.Sm + lv.p_w, lv.out_f, lv.in_f, 64)) return fail_plan();
                if (tma_out_ok(b, lv.in_f, 1)) {
                    if (!act_map(&um.dgrad.mapC, lv.d_below, B, 1, 1, lv.in_f, 1, 1, 128)) return fail_plan();
                    p.tma_out = 1;
                }
                um.dgrad.enabled = true;
            }
            // ---- weight gradient: dW_j = dY_j^T X ; M tiles enumerated per shard (needs 16-byte aligned shard starts) ----
            bool aligned = true;
            for (int j = 0; j <= K; ++j) aligned = aligned && ((((long)j * lv.out_f) / K) % 8 == 0);
            if (aligned) {
                OpBlock* b = blk(um.wgrad);
                memset(b, 0, sizeof(*b));
                UmmaParams& p = b->p;
                p.mode = MODE_WGRAD; p.ntaps = 1; p.bw = 1; p.bh = 1; p.bn = 64; p.W = 1; p.H = 1; p.N = B;
                p.tiles_w = 1; p.tiles_h = 1; p.tiles_n = cdiv_i(B, 64);
                p.total_chunks = p.tiles_n;
                p.w_cols = lv.in_f; p.n_total = lv.in_f; p.shards = 1; p.tiles_per_shard = 1;
                p.m_total = lv.out_f; p.m_shards = K; p.m_tiles_per_shard = cdiv_i(cdiv_i(lv.out_f, K), 128);
                p.tap_group = 1;
                b->bn = lv.in_f >= 256 ? 256 : (lv.in_f >= 128 ? 128 : 64);
                const int n_tiles = cdiv_i(lv.in_f, b->bn);
                p.splits = 1; p.chunks_per_split = p.total_chunks;
                p.stages = p.total_chunks < 4 ? p.total_chunks : 4;
                if (bwd_cohabit() && p.stages > cohabit_stages(b->bn)) p.stages = cohabit_stages(b->bn);
                p.epi = UEPI_F32; p.ldc = lv.in_f; p.split_stride = 0;
                p.bias_fused = 1; p.bias_off = (long)lv.n_w;
                p.out = (void*)(mv.Gm + lv.p_w);
                p.status = mv.status;
                b->grid = dim3((unsigned)(p.m_tiles_per_shard * K), (unsigned)n_tiles, 1);
                if (!act_map(&um.wgrad.mapA, lv.dact, B, 1, 1, lv.out_f, 1, 1, 64)) return fail_plan();
                if (!act_map(&um.wgrad.mapB, lv.in_act, B, 1, 1, lv.in_f, 1, 1, 64)) return fail_plan();
                // float maps over the master weights and the momentum buffer, for the weight gradient with the update folded in
                b->upd_maps = (mv.Vm != nullptr && (lv.p_w & 3) == 0 && lv.in_f % 4 == 0 &&
                               mat_map_f32(&um.wgrad.mapC, mv.Wm + lv.p_w, lv.out_f, lv.in_f) &&
                               mat_map_f32(&um.wgrad.mapD, mv.Vm + lv.p_w, lv.out_f, lv.in_f)) ? 1 : 0;
                um.wgrad.enabled = true;
            }
        }
    }
    return SB_OK;
}

sb_status umma_bind_input(sb_model* m, const void* x)
{
    ModelView mv = model_view(m);
    LayerView lv = layer_view(m, 0);
    UmmaLayer& um = *lv.um;
    if (um.bound_input == x) return SB_OK;
    if (um.fwd.enabled && !act_map(&um.fwd.mapA, x, mv.B, 1, 1, lv.in_f, 1, 1, 128)) return SB_ERR_CUDA;
    if (um.wgrad.enabled && !act_map(&um.wgrad.mapB, x, mv.B, 1, 1, lv.in_f, 1, 1, 64)) return SB_ERR_CUDA;
    um.bound_input = x;
    return SB_OK;
}

sb_status umma_conv_fwd(sb_model* m, int layer, cudaStream_t st) { return launch_op(layer_view(m, layer).um->fwd, st, launch_counter(m)); }
sb_status umma_conv_dgrad(sb_model* m, int layer, cudaStream_t st) { return launch_op(layer_view(m, layer).um->dgrad, st, launch_counter(m)); }
sb_status umma_fc_fwd(sb_model* m, int layer, cudaStream_t st) { return launch_op(layer_view(m, layer).um->fwd, st, launch_counter(m)); }
sb_status umma_fc_dgrad(sb_model* m, int layer, cudaStream_t st) { return launch_op(layer_view(m, layer).um->dgrad, st, launch_counter(m)); }
sb_status umma_fc_wgrad(sb_model* m, int layer, cudaStream_t st) { return launch_op(layer_view(m, layer).um->wgrad, st); }

bool umma_fc_wgrad_can_update(sb_model* m, int layer)
{
    const LayerView lv = layer_view(m, layer);
    if (!lv.um->wgrad.enabled) return false;
    const OpBlock* b = blk(lv.um->wgrad);
    // (the parameter arenas share the gradient arena's element offsets: 16-byte alignment of `out` carries over)
    const long smem = (long)b->p.stages * (A_STAGE_BYTES + b->bn * 128) + 1024 + CTRL_BYTES + UPD_EXTRA_SMEM;
    // (not for grids of a few dozen CTAs: the kernel holds a whole SM's shared memory per CTA -- measured per step: 4096 x 4096
    // (512 CTAs) -3.4 %, 512 -> 4096 (64 CTAs) a further -1.4 %, a 1024 x 1024 layer (32 CTAs) +0.5 %)
    static const long min_ctas = (long)tune("SB_FC_UPDATE_MIN_CTAS", 64);
    return b->p.mode == MODE_WGRAD && b->upd_maps && !b->pair && b->p.ntaps == 1 && b->bn != 192 && b->p.splits == 1 && b->p.bias_fused && wgrad_sweep_ok(b) &&
           (lv.p_w & 3) == 0 && (lv.in_f % 64) == 0 && smem <= 227 * 1024 && (long)b->grid.x * b->grid.y * b->grid.z >= min_ctas;
}
sb_status umma_fc_wgrad_update(sb_model* m, int layer, float lr, float mu, cudaStream_t st)
{
    const ModelView mv = model_view(m);
    const LayerView lv = layer_view(m, layer);
    SgdFuse f{mv.Wm + lv.p_w, mv.Vm + lv.p_w, mv.Sm ? mv.Sm + lv.p_w : nullptr, lr, mu};
    return launch_op(lv.um->wgrad, st, nullptr, &f);
}

bool umma_wgrad_bias_fused(sb_model* m, int layer)
{
    const UmmaLayer& um = *layer_view(m, layer).um;
    return um.wgrad.enabled && blk(um.wgrad)->p.bias_fused != 0;
}

sb_status umma_conv_wgrad_launch(sb_model* m, int layer, cudaStream_t st, int* splits, float** part)
{
    LayerView lv = layer_view(m, layer);
    const OpBlock* b = blk(lv.um->wgrad);
    *splits = b->p.splits;
    *part = (float*)b->p.out;
    return launch_op(lv.um->wgrad, st);
}

}  // namespace sb
