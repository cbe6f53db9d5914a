/* Graph record of the CPU oracle (test infrastructure only; see moc_oracle.c). */
#ifndef MOC_ORACLE_GRAPH_H_
#define MOC_ORACLE_GRAPH_H_
#include <stdint.h>

typedef struct {
    int32_t n;
    int32_t C;
    int64_t n_edges;
    int64_t *pred_start; /* n+1 */
    int32_t *pred;       /* n_edges, grouped by consumer */
    uint8_t *has_succ;   /* n */
    int64_t *w, *m;      /* n */
    int32_t *cap;        /* n per-node caps C_v, or NULL: every node may have C copies */
} ograph;

#endif
