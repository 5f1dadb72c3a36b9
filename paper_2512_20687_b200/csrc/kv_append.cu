// KV-cache append: the cache half of the streaming update STEP (Eq. 12, Eq. 13).
// A bit copy of n_rows new rows per unit plus the length update.
#include "common.cuh"
#include "ptx.cuh"

// One CTA per appended item.  Every thread reads len[u] before the CTA-wide
// barrier and only thread 0 writes it after, and unit ids within a call are
// distinct, so no thread can observe the updated length.  Index arrays are read
// through the L2 (another kernel may have written them just before).  The kernel
// lets its successor start at once: the attention that follows reads lengths and
// pages through the L2 only and touches no key or value before its own
// dependency wait, so all it does early is its set-up.
__global__ void __launch_bounds__(128)
kv_append_kernel(uint4 *__restrict__ k, uint4 *__restrict__ v, int32_t *__restrict__ len, int n_units,
                 int Hkv, int cap, int vec_per_row, const uint4 *__restrict__ k_new,
                 const uint4 *__restrict__ v_new, const int32_t *__restrict__ unit_ids, int n_rows,
                 const Paging pg, int32_t *__restrict__ status) {
    const int i = blockIdx.x;
    ptx::grid_dep_launch();
    ptx::grid_dep_wait();
    const int u = unit_ids ? __ldcg(unit_ids + i) : i;
    if (u < 0 || u >= n_units) {
        if (threadIdx.x == 0) atomicOr(status, PHOTON_DEV_BAD_INDEX);
        return;
    }
    const int at = __ldcg(len + u);
    if (at < 0 || at + n_rows > cap) {
        if (threadIdx.x == 0) atomicOr(status, PHOTON_DEV_CAPACITY);
        return;
    }
    const int per_item = n_rows * Hkv * vec_per_row;
    if (pg.table) {
        // a paged cache: every page the new rows fall into must exist before anything is written
        for (int r = at / pg.page_rows; r <= (at + n_rows - 1) / pg.page_rows; ++r) {
            const int id = __ldcg(pg.table + (size_t)u * pg.pages_per_unit + r);
            if (id < 0 || id >= pg.n_pages) {
                if (threadIdx.x == 0) atomicOr(status, PHOTON_DEV_BAD_INDEX);
                return;
            }
        }
    }
    for (int t = threadIdx.x; t < per_item; t += blockDim.x) {
        const int d = t % vec_per_row;
        const int h = (t / vec_per_row) % Hkv;
        const int r = t / (vec_per_row * Hkv);
        const size_t src = (size_t)i * per_item + t;      // [n, n_rows, Hkv, dh]
        size_t dst;
        if (pg.table) {
            const int row = at + r;
            const int id = __ldcg(pg.table + (size_t)u * pg.pages_per_unit + row / pg.page_rows);
            dst = (((size_t)id * Hkv + h) * pg.page_rows + row % pg.page_rows) * vec_per_row + d;
        } else {
            dst = (((size_t)u * Hkv + h) * cap + (at + r)) * vec_per_row + d;
        }
        k[dst] = k_new[src];
        v[dst] = v_new[src];
    }
    __syncthreads();
    if (threadIdx.x == 0) len[u] = at + n_rows;
}

cudaError_t launch_kv_append(bf16 *k, bf16 *v, int32_t *len, int n_units, int Hkv, int cap, int dh,
                             const bf16 *k_new, const bf16 *v_new, const int32_t *unit_ids, int n,
                             int n_rows, Paging pg, int32_t *status, cudaStream_t st, long long *launches) {
    if (n == 0) return cudaSuccess;
    const cudaError_t e = launch_dependent(kv_append_kernel, dim3(n), dim3(128), 0, st, 0, (uint4 *)k, (uint4 *)v, len, n_units, Hkv, cap, dh / 8,
                                        (const uint4 *)k_new, (const uint4 *)v_new, unit_ids, n_rows,
                                        pg, status);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}
