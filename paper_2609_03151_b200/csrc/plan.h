// Internal definition of the opaque plan object (host only).
#pragma once
#include "basp.h"

struct basp_plan {
    basp_config cfg;
    int N, B, G, K, Bl, S, T;
    int Hq, Hkv, D;
    int Hq_l, Hkv_l;   // heads per rank after the first all-to-all
    int kv_rep;        // ranks of a group that hold the same KV head (1 unless the group has more ranks than KV heads)
    int causal;
};

// Thread-local CUDA error text shared by the translation units.
void basp_set_cuda_error(const char *what, int cuda_code, const char *text);
void basp_count_launch(int n);
