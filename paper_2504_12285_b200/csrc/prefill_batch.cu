// Grouped prefill: several BitLinear forwards of more than 16 tokens each in three launches.
// (Paper Section 5.1: packed weights are expanded on chip to a form the matrix units consume, then multiplied with
// the 8-bit activations; here the expansion and the activation quantiser write directly the shared-memory images of
// the tensor-core kernel's tiles, and one persistent kernel runs the tiles of every matmul of the group.)
//
//   launch 1  group_unpack_kernel : packed 2-bit weights -> byte codes in 256 x 128 tile images, with a count of
//                                   finished words per 256-row weight tile.
//   launch 2  group_quant_warp_kernel : one warp per token - fused RMSNorm + absmax int8 quantiser; codes go into
//                                   128 x 128 tile images (128-byte swizzle) of the activation operand.  Problems
//                                   that read the same activations share one quantised copy.  Starts as a
//                                   programmatic dependent of launch 1 and runs beside it (no shared data).
//   launch 3  gemm_i8_pair_kernel : every tile of every matmul on CTA pairs (gemm_i8_kernel<true> when the SMs do not
//                                   pair up), operands fetched as whole tile images.  The pair kernel is a
//                                   programmatic dependent too: it waits for launch 2 as a whole
//                                   (griddepcontrol.wait) and for launch 1 tile by tile (the word counts).
// Problems are ordered by decreasing K so that the long tiles are scheduled first and the tail is made of short ones,
// after the small matrices, whose tiles can start while the large ones are still being expanded.
#include <algorithm>
#include <vector>

#include "quant_row.cuh"

namespace bitlinear {

namespace {

struct PrefillItem {
    const void* x;  // first operand of the input step (see RowOp)
    RowOp op;       // the element-wise step in front of the quantiser
    const __nv_bfloat16* gain;
    const uint32_t* packed;
    uint8_t* a_tiles;
    uint8_t* codes;
    float* d;
    int32_t* xsum;
    long long word_begin;  // packed 32-bit words of the problems before this one
    float eps;
    int M, N, K;
    int row_begin;  // tokens of the problems before this one
    int nt_begin;   // 256-row weight tiles of the problems before this one
};
constexpr size_t kItemTableBytes = kMaxGroup * sizeof(PrefillItem);

// One warp per token, eight tokens per CTA.
__global__ void __launch_bounds__(kQuantThreads) group_quant_warp_kernel(const PrefillItem* __restrict__ items, int count,
                                                                         int rows) {
    // This launch runs beside the expansion launch before it (it reads nothing of it), and the GEMM launch after it
    // may start: it waits for this grid with griddepcontrol.wait before it reads anything written here.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int row = blockIdx.x * kQuantWarps + (threadIdx.x >> 5);
    if (row >= rows) return;
    int i = 0;
    while (i + 1 < count && row >= items[i + 1].row_begin) ++i;
    const PrefillItem& p = items[i];
    const int m = row - p.row_begin;
    uint8_t* dst = p.a_tiles + (size_t)(m >> 7) * (p.K >> 7) * (128 * 128) + (size_t)(m & 127) * 128;
    with_row_source(p.op, p.x, m, p.K, [&](auto src) {
        quant_row_warp_src<2>(src, p.gain, p.eps, p.K, reinterpret_cast<int8_t*>(dst), p.d + m, p.xsum + m, m & 7);
    });
}

// Expansion of the packed weights into tile images: one thread per packed word (16 codes -> its 16-byte piece of a
// 256 x 128 image), persistent CTAs that walk the words of all problems in table order, 2,048 words at a time.  After
// every step the CTA adds its words to the ready counter of the 256-row weight tile they belong to: the GEMM kernel,
// which starts beside this launch and consumes the tiles in the same order, reads a tile's images as soon as all its
// words are counted.  (A weight tile has 16 * K words, the last one of a matrix 8 * K: multiples of 2,048 for every
// valid shape - N a multiple of 128, K of 256 - so a step never straddles two tiles.)
constexpr int kUnpackChunk = 2048;  // packed words per CTA step: 8 per thread, all loaded before anything is stored
__global__ void __launch_bounds__(256) group_unpack_kernel(const PrefillItem* __restrict__ items, int count,
                                                           long long total_words, int* __restrict__ ready) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int i = 0;
    for (long long chunk = (long long)blockIdx.x * kUnpackChunk; chunk < total_words; chunk += (long long)gridDim.x * kUnpackChunk) {
        while (i + 1 < count && chunk >= items[i + 1].word_begin) ++i;
        const PrefillItem& p = items[i];
        const int k_tiles = p.K / kTileCols;
        const size_t w0 = (size_t)(chunk - p.word_begin) + threadIdx.x;
        uint32_t v[kUnpackChunk / 256];
#pragma unroll
        for (int u = 0; u < kUnpackChunk / 256; ++u) v[u] = p.packed[w0 + (size_t)u * 256];
#pragma unroll
        for (int u = 0; u < kUnpackChunk / 256; ++u) {
            const size_t w = w0 + (size_t)u * 256;
            // position of packed word w (see "Packed weight layout" in bitlinear.h)
            const size_t tile = w >> 8;
            const int wo = (int)(w & 255);
            const int h = wo >> 7, g = (wo >> 4) & 7, t = (wo >> 2) & 3, q = wo & 3;
            const int n = (int)(tile / k_tiles) * kTileRows + 8 * h + g;
            const int k0 = (int)(tile % k_tiles) * kTileCols + 64 * t + 16 * q;
            const int r = n & 255, piece = (k0 & 127) >> 4;
            const size_t img = (size_t)(n >> 8) * (p.K / 128) + (k0 >> 7);
            *reinterpret_cast<uint4*>(p.codes + img * 32768 + (size_t)r * 128 + ((piece ^ (r & 7)) << 4)) =
                make_uint4(v[u] & 0x03030303u, (v[u] >> 2) & 0x03030303u, (v[u] >> 4) & 0x03030303u, (v[u] >> 6) & 0x03030303u);
        }
        __syncthreads();  // every store of the chunk is ordered before the fence and the count below
        if (threadIdx.x == 0) {
            __threadfence();
            // the step lies inside one 256-row weight tile (16 * K words each)
            atomicAdd(ready + p.nt_begin + (int)((chunk - p.word_begin) / (16 * (long long)p.K)), kUnpackChunk);
        }
    }
}

struct GroupLayout {
    size_t table_off, items_off, ready_off, ready_bytes, total;
    std::vector<size_t> a_off, codes_off, d_off, xsum_off;
};

GroupLayout group_layout(const bitlinear_problem* problems, const int* idx, int n) {
    GroupLayout L;
    size_t off = 0;
    L.table_off = off;
    off = align_up(off + kGroupTableDevBytes, 256);
    L.items_off = off;
    off = align_up(off + kItemTableBytes, 256);
    L.ready_off = off;
    size_t n_tiles = 0;
    for (int i = 0; i < n; ++i) n_tiles += (size_t)(problems[idx[i]].N + 255) / 256;
    L.ready_bytes = align_up(n_tiles * sizeof(int), 256);
    off = align_up(off + L.ready_bytes, 1024);
    for (int i = 0; i < n; ++i) {
        const bitlinear_problem& q = problems[idx[i]];
        L.a_off.push_back(off);
        off = align_up(off + gemm_a_tiles_bytes(q.M, q.K), 1024);
        L.codes_off.push_back(off);
        off = align_up(off + gemm_codes_bytes(q.N, q.K), 1024);
        L.d_off.push_back(off);
        off = align_up(off + (size_t)q.M * sizeof(float), 1024);
        L.xsum_off.push_back(off);
        off = align_up(off + (size_t)q.M * sizeof(int32_t), 1024);  // every piece a multiple of 1 KiB: the total does not depend on the order
    }
    L.total = off;
    return L;
}

}  // namespace

// Workspace of a group of prefill problems (problems[idx[0..n)], every M > 16); at most kMaxGroup per launch group,
// larger sets are run as consecutive groups over the same layout.
size_t prefill_group_workspace_bytes(const bitlinear_problem* problems, const int* idx, int n) {
    size_t total = 0;
    for (int b = 0; b < n; b += kMaxGroup) total += group_layout(problems, idx + b, std::min(kMaxGroup, n - b)).total;
    return total;
}

int prefill_group_forward(const bitlinear_problem* problems, const int* idx_in, int n_in, void* ws, bool skip_quant,
                          bool skip_unpack, cudaStream_t st) {
    char* base_all = static_cast<char*>(ws);
    int sm_count = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        sm_count <= 0) {
        cudaGetLastError();
        return BITLINEAR_ERR_CUDA;
    }
    for (int b = 0; b < n_in; b += kMaxGroup) {
        const int n = std::min(kMaxGroup, n_in - b);
        std::vector<int> idx(idx_in + b, idx_in + b + n);
        // Where the SMs pair up the GEMM reads the packed weights themselves and expands them in shared memory: no
        // expansion launch, no code images.  (Otherwise: expansion launch + single-CTA kernel on the code images.)
        const bool in_kernel_expansion = (sm_count % 2) == 0;
        if (in_kernel_expansion) {
            // One persistent kernel walks the tiles of all problems in table order, CTA pair p taking tiles p, p + pairs, ...
            // Problems that share an input stay together, small ones first; and the schedule must not END on the longest
            // tiles (its last, partly filled wave costs a whole tile time): if the last problem has the largest K, the
            // latest problem with a smaller K goes behind it.  (Measured on the 7 shapes of a layer at 2,048 tokens:
            // 113 us against 115-117 us in order of decreasing K.)
            auto first_user = [&](int i) {  // the first problem of the call that names the same input
                for (int j : idx)
                    if (problems[j].x == problems[i].x && problems[j].x2 == problems[i].x2 && problems[j].M == problems[i].M &&
                        problems[j].K == problems[i].K)
                        return j;
                return i;
            };
            std::vector<int> order(idx.size()), group_of(idx.size());
            for (size_t a = 0; a < idx.size(); ++a) order[a] = (int)a, group_of[a] = first_user(idx[a]);
            std::stable_sort(order.begin(), order.end(), [&](int l, int r) {
                const bitlinear_problem &pl = problems[idx[l]], &pr = problems[idx[r]];
                const long long cl = (long long)pl.M * pl.K, cr = (long long)pr.M * pr.K;
                if (cl != cr) return cl < cr;
                if (group_of[l] != group_of[r]) return group_of[l] < group_of[r];
                return (long long)pl.N * pl.K < (long long)pr.N * pr.K;
            });
            std::vector<int> sorted;
            for (int a : order) sorted.push_back(idx[a]);
            idx = sorted;
            const int k_last = problems[idx.back()].K;
            bool largest = true;
            for (int i : idx) largest = largest && problems[i].K <= k_last;
            if (largest) {
                for (int a = (int)idx.size() - 2; a >= 0; --a)
                    if (problems[idx[a]].K < k_last) {
                        const int moved = idx[a];
                        idx.erase(idx.begin() + a);
                        idx.push_back(moved);
                        break;
                    }
            }
        } else {
            std::stable_sort(idx.begin(), idx.end(), [&](int l, int r) { return problems[l].K > problems[r].K; });
            // ... except that small matrices go first: their codes are expanded within a microsecond, so the GEMM's first
            // tiles start at once while the expansion of the large matrices runs ahead of the tiles that need them
            size_t largest = 0;
            for (int i : idx) largest = std::max(largest, (size_t)problems[i].N * problems[i].K);
            std::stable_partition(idx.begin(), idx.end(), [&](int i) { return (size_t)problems[i].N * problems[i].K * 4 <= largest; });
        }
        const GroupLayout L = group_layout(problems, idx.data(), n);
        char* base = base_all;
        base_all += L.total;

        PrefillItem items[kMaxGroup] = {};
        GemmProblem gp[kMaxGroup] = {};
        const void* packed_ptrs[kMaxGroup] = {};
        if (in_kernel_expansion) skip_unpack = true;
        long long words = 0;
        int rows = 0, nt_total = 0;
        for (int i = 0; i < n; ++i) {
            const bitlinear_problem& q = problems[idx[i]];
            PrefillItem& it = items[i];
            it.x = q.x;
            it.op.x2 = q.x2; it.op.x_out = q.x_out; it.op.op = q.x_op; it.op.arg0 = q.x_arg0; it.op.arg1 = q.x_arg1; it.op.pad = 0;
            it.gain = static_cast<const __nv_bfloat16*>(q.gain);
            it.packed = static_cast<const uint32_t*>(q.packed);
            it.a_tiles = reinterpret_cast<uint8_t*>(base + L.a_off[i]);
            it.codes = reinterpret_cast<uint8_t*>(base + L.codes_off[i]);
            it.d = reinterpret_cast<float*>(base + L.d_off[i]);
            it.xsum = reinterpret_cast<int32_t*>(base + L.xsum_off[i]);
            it.word_begin = words;
            it.eps = q.rms_eps;
            it.M = q.M; it.N = q.N; it.K = q.K;
            it.row_begin = rows;
            it.nt_begin = nt_total;
            nt_total += (q.N + 255) / 256;
            words += (long long)q.N * q.K / 16;
            // problems that read the same activations (q/k/v, gate/up of a layer) share one quantised copy
            int same = -1;
            for (int j = 0; j < i && same < 0; ++j) {
                const bitlinear_problem& o = problems[idx[j]];
                if (o.x == q.x && o.x2 == q.x2 && o.x_op == q.x_op && o.x_out == q.x_out && o.x_arg0 == q.x_arg0 &&
                    o.x_arg1 == q.x_arg1 && o.gain == q.gain && o.rms_eps == q.rms_eps && o.M == q.M && o.K == q.K)
                    same = j;
            }
            if (same >= 0) {
                it.a_tiles = items[same].a_tiles; it.d = items[same].d; it.xsum = items[same].xsum;
            } else {
                rows += q.M;
            }
            packed_ptrs[i] = q.packed;
            GemmProblem& g = gp[i];
            g.a_tiles = it.a_tiles; g.codes = it.codes; g.d = it.d; g.xsum = it.xsum; g.s_w = q.s_w;
            g.y = q.y; g.acc_out = nullptr;
            g.M = q.M; g.N = q.N; g.K = q.K; g.y_dtype = q.y_dtype;
        }
        PrefillItem* items_dev = reinterpret_cast<PrefillItem*>(base + L.items_off);
        int* ready = reinterpret_cast<int*>(base + L.ready_off);
        if (cudaMemsetAsync(ready, 0, L.ready_bytes, st) != cudaSuccess ||
            cudaMemcpyAsync(items_dev, items, sizeof(PrefillItem) * n, cudaMemcpyHostToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return BITLINEAR_ERR_CUDA;
        }
        // The quantiser and expansion launches go between the GEMM's table upload and the GEMM kernel, which starts
        // as a programmatic dependent of the expansion launch and follows it problem by problem.
        struct Launches {
            const PrefillItem* items_dev;
            int* ready;
            int n, rows, sm_count;
            long long words;
            bool skip_quant, skip_unpack;
            cudaStream_t st;
            static int run(void* ctx) {
                const Launches& a = *static_cast<const Launches*>(ctx);
                // the expansion first (at most four CTAs per SM, so that the other kernels find room beside them) ...
                if (!a.skip_unpack) {
                    const long long chunks = (a.words + kUnpackChunk - 1) / kUnpackChunk;
                    const unsigned grid = (unsigned)std::min<long long>(chunks, 4LL * a.sm_count);
                    group_unpack_kernel<<<grid, 256, 0, a.st>>>(a.items_dev, a.n, a.words, a.ready);
                    if (cudaGetLastError() != cudaSuccess) return (int)BITLINEAR_ERR_CUDA;
                }
                if (a.skip_quant) return (int)BITLINEAR_OK;
                if (a.skip_unpack) {  // nothing to run beside: an ordinary launch, the GEMM after it is ordinary too
                    group_quant_warp_kernel<<<(unsigned)((a.rows + kQuantWarps - 1) / kQuantWarps), kQuantThreads, 0, a.st>>>(
                        a.items_dev, a.n, a.rows);
                    return cudaGetLastError() == cudaSuccess ? (int)BITLINEAR_OK : (int)BITLINEAR_ERR_CUDA;
                }
                // ... then the quantiser as its programmatic dependent: the two share no data and run side by side
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3((unsigned)((a.rows + kQuantWarps - 1) / kQuantWarps));
                cfg.blockDim = dim3(kQuantThreads);
                cfg.stream = a.st;
                cudaLaunchAttribute attr[1];
                attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
                attr[0].val.programmaticStreamSerializationAllowed = 1;
                cfg.attrs = attr;
                cfg.numAttrs = 1;
                if (cudaLaunchKernelEx(&cfg, group_quant_warp_kernel, a.items_dev, a.n, a.rows) != cudaSuccess) {
                    cudaGetLastError();
                    return (int)BITLINEAR_ERR_CUDA;
                }
                return (int)BITLINEAR_OK;
            }
        } launches = {items_dev, ready, n, rows, sm_count, words, skip_quant, skip_unpack, st};
        // with the expanded codes of an earlier call still in place there is nothing to follow tile by tile: the GEMM is
        // then an ordinary launch behind the quantiser (or behind nothing)
        const int rc = gemm_launch(gp, n, true, nullptr, reinterpret_cast<uint8_t*>(base + L.table_off), st, base, L.total,
                                   skip_unpack ? nullptr : ready, &Launches::run, &launches, /*wait_primary=*/!skip_quant,
                                   /*a_ready=*/nullptr, in_kernel_expansion ? packed_ptrs : nullptr);
        if (rc != BITLINEAR_OK) return rc;
    }
    return BITLINEAR_OK;
}

}  // namespace bitlinear
