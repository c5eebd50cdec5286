/*
 * CPU ORACLE -- TEST INFRASTRUCTURE ONLY.  Not part of the product path; shares no code
 * with the CUDA library.
 *
 * Shortest-path-distance (SPD) index matrix of one graph, the structural encoding that
 * selects the additive attention bias (the paper's "structural encoding ... such as
 * shortest path distances", Sec. Preliminaries and Sec. Graph-Aware Context Parallelism,
 * item 2).
 *
 * Definition implemented, exactly:  for every source s, textbook queue BFS over the CSR
 * out-neighbour lists until the queue is empty;
 *     spd[s][t] = min(hops(s -> t), max_dist)   if t is reachable from s
 *               = max_dist + 1                  otherwise,
 * spd[s][s] = 0.  Reachable pairs farther than max_dist are clipped to max_dist and stay
 * distinct from unreachable pairs, so the traversal is never cut short.
 * Padding bytes (columns n .. ld-1 of every row) are set to 255.
 *
 * Sources are independent; the only parallelism is an OpenMP loop over them.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* Rows of the SPD matrix for the listed sources only: row i of `spd` (pitch ld) is the full
 * distance row of source sources[i].  sources == NULL means all n sources in order. */
int oracle_spd_bfs_sources(int32_t n, const int32_t* row_ptr, const int32_t* col_idx,
                           int32_t max_dist, int64_t ld, int32_t n_sources, const int32_t* sources,
                           uint8_t* spd)
{
    if (n < 0 || max_dist < 1 || max_dist > 254 || ld < n || n_sources < 0) return 1;
    int fail = 0;
#pragma omp parallel
    {
        int32_t* dist  = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
        int32_t* queue = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
        if (!dist || !queue) {
#pragma omp atomic write
            fail = 1;
        } else {
#pragma omp for schedule(dynamic, 16)
            for (int32_t si = 0; si < n_sources; ++si) {
                const int32_t s = sources ? sources[si] : si;
                for (int32_t t = 0; t < n; ++t) dist[t] = -1;
                int32_t head = 0, tail = 0;
                dist[s] = 0;
                queue[tail++] = s;
                while (head < tail) {
                    int32_t u = queue[head++];
                    for (int32_t e = row_ptr[u]; e < row_ptr[u + 1]; ++e) {
                        int32_t w = col_idx[e];
                        if (dist[w] < 0) {
                            dist[w] = dist[u] + 1;
                            queue[tail++] = w;
                        }
                    }
                }
                uint8_t* row = spd + (int64_t)si * ld;
                for (int32_t t = 0; t < n; ++t) {
                    int32_t dd = dist[t];
                    row[t] = (uint8_t)(dd < 0 ? max_dist + 1 : (dd > max_dist ? max_dist : dd));
                }
                for (int64_t t = n; t < ld; ++t) row[t] = 255;
            }
        }
        free(dist);
        free(queue);
    }
    return fail ? 2 : 0;
}

int oracle_spd_bfs(int32_t n, const int32_t* row_ptr, const int32_t* col_idx,
                   int32_t max_dist, int64_t ld, uint8_t* spd)
{
    return oracle_spd_bfs_sources(n, row_ptr, col_idx, max_dist, ld, n, (const int32_t*)0, spd);
}
