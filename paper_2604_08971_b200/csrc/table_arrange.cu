// Sample-table preparation for SentryAttend's sparsity score (Section 4.4).  The score of query i
// is taken over a fixed set S_i of sampled key positions; the ORDER in which a kernel visits the
// members of S_i is free.  The score kernels give one query to one thread and keep the group's key
// rows in shared memory, so a warp's 32 threads read 32 key rows at unrelated positions at every
// step, eight threads per shared-memory access phase, and rows whose index is equal modulo 8 fall
// on the same banks (for every supported head dimension the bank group of a 16-byte piece of row r
// is a function of r mod 8 and the piece number).  With the members of S_i in arbitrary order a
// phase meets 2.6 rows per bank group on average.
//
// This kernel writes the tables entry-major (what score_mode 2 reads: sample j of query i at
// j * T_v + i) and, for every block of 8 consecutive queries, orders the members of each S_i so
// that the 8 rows read at the same step have distinct indices modulo 8 wherever that is possible:
// step by step, a maximum bipartite matching between the 8 queries and the 8 residues they still
// have unused members of.  Random tables come out at ~1.35 rows per bank group; the sets are
// unchanged.
#include "common.cuh"

namespace {

constexpr int kArrThreads = 128;
constexpr int kArrMaxSamples = 64;   // members per set the used-mask can hold

// One block per mask value s; thread g arranges queries 8g .. 8g+7 of that subset's table.
__global__ void __launch_bounds__(kArrThreads)
table_arrange_kernel(const int32_t* __restrict__ ids, int Tlen, int c, const int32_t* __restrict__ table,
                     const int64_t* __restrict__ offsets, int32_t* __restrict__ out, unsigned int* status) {
    __shared__ int red[33];
    const uint32_t s = blockIdx.x;
    const long long off = offsets[s];
    if (off < 0) return;
    int mine = 0;
    for (int t = threadIdx.x; t < Tlen; t += blockDim.x) {
        const int m = ids[t];
        mine += (m >= 0 && m < 32 && ((s >> m) & 1u)) ? 1 : 0;
    }
    const int Tv = block_sum_int(mine, red);
    if (Tv == 0) return;
    const int n_s = sentry_num_active(Tv, c);
    if (n_s > kArrMaxSamples) {   // the host checks U(T) <= kArrMaxSamples
        if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
        return;
    }
    const int32_t* tbl = table + off;
    int32_t* dst = out + off;
    for (int g = threadIdx.x; g * 8 < Tv; g += blockDim.x) {
        const int q0 = g * 8, nq = min(8, Tv - q0);
        unsigned long long used[8];
        unsigned char cnt[8][8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            used[q] = 0ull;
#pragma unroll
            for (int r = 0; r < 8; ++r) cnt[q][r] = 0;
        }
        for (int q = 0; q < nq; ++q)
            for (int j = 0; j < n_s; ++j) {
                int v = tbl[(size_t)(q0 + q) * n_s + j];
                if (v < 0 || v >= Tv) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); v = 0; }
                ++cnt[q][v & 7];
            }
        for (int a = 0; a < n_s; ++a) {
            // maximum matching queries -> residues (augmenting paths, breadth first)
            int match_q[8], match_r[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) { match_q[i] = -1; match_r[i] = -1; }
            for (int q = 0; q < nq; ++q) {
                int from_q[8], queue[8];
                int head = 0, tail = 0;
                unsigned seen = 0u;
                queue[tail++] = q;
                bool done = false;
                while (head < tail && !done) {
                    const int x = queue[head++];
                    for (int r = 0; r < 8 && !done; ++r) {
                        if (cnt[x][r] == 0 || ((seen >> r) & 1u)) continue;
                        seen |= 1u << r;
                        from_q[r] = x;
                        if (match_r[r] < 0) {
                            int rc = r;
                            for (;;) {   // flip the path back to q
                                const int qx = from_q[rc];
                                const int prev = match_q[qx];
                                match_r[rc] = qx;
                                match_q[qx] = rc;
                                if (qx == q) break;
                                rc = prev;
                            }
                            done = true;
                        } else {
                            queue[tail++] = match_r[r];
                        }
                    }
                }
            }
            // every query places one unused member: of its matched residue, else the first unused
            for (int q = 0; q < nq; ++q) {
                const int want = match_q[q];
                int pick = -1, pick_v = 0;
                for (int j = 0; j < n_s; ++j) {
                    if ((used[q] >> j) & 1ull) continue;
                    int v = tbl[(size_t)(q0 + q) * n_s + j];
                    if (v < 0 || v >= Tv) v = 0;
                    if (want < 0 || (v & 7) == want) { pick = j; pick_v = v; break; }
                }
                used[q] |= 1ull << pick;
                --cnt[q][pick_v & 7];
                dst[(size_t)a * Tv + q0 + q] = pick_v;
            }
        }
    }
}

}  // namespace

int launch_table_arrange(sentry_ctx* ctx, const int32_t* ids, int T, int c, const int32_t* table,
                         const int64_t* offsets, int n_subsets, int32_t* out, cudaStream_t st) {
    if (sentry_num_active(T, c) > kArrMaxSamples) return SENTRY_ERR_UNSUPPORTED;
    LaunchScope ls(ctx, KS_TABLE_ARRANGE, st);
    table_arrange_kernel<<<n_subsets, kArrThreads, 0, st>>>(ids, T, c, table, offsets, out, ctx->d_status);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}
