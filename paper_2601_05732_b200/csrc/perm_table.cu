// Permutation tables of the Birkhoff-von Neumann parameterisation (paper Theorem 3.1, Section 3.2).
//
// sigma[k][i] lists the n! permutations of (0..n-1) in lexicographic order (k = 0 is the identity);
// P_k[i][sigma_k(i)] = 1, so H_res[i][j] = sum of a_k over the (n-1)! permutations with sigma_k(i) = j.
// klist stores, for every entry (i,j), those (n-1)! indices k in increasing order.
#include "common.cuh"

namespace mhcl {

__constant__ PermTables c_perm[kMaxN + 1];

// Successor in lexicographic order; returns false after the last permutation.
static bool next_lex(uint8_t* p, int n) {
    int i = n - 2;
    while (i >= 0 && p[i] > p[i + 1]) --i;          // longest non-increasing suffix
    if (i < 0) return false;
    int j = n - 1;
    while (p[j] < p[i]) --j;                        // rightmost element larger than the pivot
    uint8_t t = p[i]; p[i] = p[j]; p[j] = t;
    for (int a = i + 1, b = n - 1; a < b; ++a, --b) { t = p[a]; p[a] = p[b]; p[b] = t; }
    return true;
}

void host_perm_tables(int n, PermTables* out) {
    memset(out, 0, sizeof(*out));
    uint8_t cur[kMaxN];
    for (int i = 0; i < n; ++i) cur[i] = (uint8_t)i;
    int k = 0;
    int fill[kMaxN * kMaxN] = {0};
    const int per = ipow_fact(n - 1);
    do {
        for (int i = 0; i < n; ++i) {
            out->sigma[k * n + i] = cur[i];
            const int e = i * n + cur[i];
            out->klist[e * per + fill[e]++] = (uint8_t)k;
        }
        ++k;
    } while (next_lex(cur, n));
}

cudaError_t upload_perm_tables(int n) {
    PermTables h;
    host_perm_tables(n, &h);
    return cudaMemcpyToSymbol(c_perm, &h, sizeof(PermTables), sizeof(PermTables) * n, cudaMemcpyHostToDevice);
}

cudaError_t download_perm_sigma(int n, uint8_t* sigma_host) {
    PermTables h;
    cudaError_t e = cudaMemcpyFromSymbol(&h, c_perm, sizeof(PermTables), sizeof(PermTables) * n, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return e;
    memcpy(sigma_host, h.sigma, (size_t)ipow_fact(n) * n);
    return cudaSuccess;
}

}  // namespace mhcl
