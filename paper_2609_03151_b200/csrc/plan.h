// Internal definition of the opaque plan object (host only).
#pragma once
#include "basp.h"

struct basp_plan {
    basp_config cfg;
    int N, B, G, K, Bl, S, T;
    int T_last;        // tokens of a group's last rank per sequence: T unless K does not divide S (then S - (K-1)*T)
    int Hq, Hkv, D;
    int Hq_l, Hkv_l;   // heads per rank after the first all-to-all
    int kv_rep;        // ranks of a group that hold the same KV head (1 unless the group has more ranks than KV heads)
    int causal;
};

// Thread-local CUDA error text shared by the translation units.
// Tokens per sequence held by local rank l (Algorithm 2's chunk, the last one short when K does not divide S).
inline int basp_rank_tokens(const basp_plan *p, int l) { return l == p->K - 1 ? p->T_last : p->T; }

void basp_set_cuda_error(const char *what, int cuda_code, const char *text);
void basp_count_launch(int n);
