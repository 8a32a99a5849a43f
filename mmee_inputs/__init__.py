"""Synthetic, deterministic inputs for the MMEE search path.

Only shapes and accelerator constants live here: attention workload tuples, accelerator
parameter sets and search options, as plain dicts whose keys are the field names of the
three input structs (workload, arch, objective).  No part of the cost model is computed in
this module; both the CUDA library's binding and the CPU oracle receive these dicts and do
their own set-up.
"""
from __future__ import annotations

import random

OBJ_ENERGY, OBJ_LATENCY, OBJ_EDP, OBJ_ENERGY_LCAP, OBJ_LATENCY_ECAP = 0, 1, 2, 3, 4
TILE_POW2, TILE_ALL_DIVISORS = 0, 1
ORD_NORECOMP2, ORD_ALL6 = 0, 1
FUSE_FUSED, FUSE_SOFTMAX_IN_OP1, FUSE_SEPARATE = 1, 2, 4
FUSE_ALL = 7

KiB = 1024
MiB = 1024 * 1024


def workload(batch, q_heads, kv_heads, seq_q, seq_kv, d_qk, d_v, word_bytes=2):
    return dict(batch=batch, q_heads=q_heads, kv_heads=kv_heads, seq_q=seq_q, seq_kv=seq_kv,
                d_qk=d_qk, d_v=d_v, word_bytes=word_bytes)


def arch(pe_rows, pe_cols, n_arrays, gb_bytes, rf_bytes, dram_words_per_cycle,
         e_dram_pj, e_gb_pj, e_rf_pj, e_mac_pj, c_softmax=10.0, energy_quantum_pj=1.0):
    return dict(pe_rows=pe_rows, pe_cols=pe_cols, n_arrays=n_arrays, gb_bytes=gb_bytes,
                rf_bytes=rf_bytes, dram_words_per_cycle=dram_words_per_cycle,
                e_dram_pj=e_dram_pj, e_gb_pj=e_gb_pj, e_rf_pj=e_rf_pj, e_mac_pj=e_mac_pj,
                c_softmax=c_softmax, energy_quantum_pj=energy_quantum_pj)


def objective(objective=OBJ_ENERGY, topk=1, tiling_set=TILE_ALL_DIVISORS, order_set=ORD_ALL6,
              fuse_mask=FUSE_ALL, t_begin=0, t_end=0, row_pruning=0, key_cap=0, stationary_mask=0, rf_tiling=0):
    return dict(objective=objective, topk=topk, tiling_set=tiling_set, order_set=order_set,
                fuse_mask=fuse_mask, row_pruning=row_pruning, t_begin=t_begin, t_end=t_end, key_cap=key_cap,
                stationary_mask=stationary_mask, rf_tiling=rf_tiling)


# --- accelerators -----------------------------------------------------------------------------

def arch_tiny():
    """8x8 PE array, DRAM + 32 KB global buffer, no register-file level."""
    return arch(8, 8, 1, 32 * KiB, 0, 64, 200.0, 6.0, 0.0, 1.0)


def arch_edge():
    """16x16 PE array, DRAM / 256 KB global buffer / 1 KB register file per PE."""
    return arch(16, 16, 1, 256 * KiB, 1 * KiB, 32, 200.0, 6.0, 1.0, 1.0)


def arch_cloud():
    """128x128 PE array, HBM / 8 MB global buffer / 2 KB register file per PE."""
    return arch(128, 128, 1, 8 * MiB, 2 * KiB, 512, 120.0, 4.0, 0.8, 0.5, energy_quantum_pj=0.1)


def arch_accel1():
    """The paper's first evaluation accelerator (Section VII-A): 4 arrays of 32x32 PEs, 1 MB buffer,
    60 GB/s DRAM at 1 GHz with 2-byte words = 30 words/cycle.  Energy constants are stand-ins."""
    return arch(32, 32, 4, 1 * MiB, 1 * KiB, 30, 200.0, 6.0, 1.0, 1.0)


# --- the five benchmark configurations --------------------------------------------------------

def config1():
    """Tiny single-head attention, power-of-two tilings, two loop orders, fuse / no-fuse."""
    return dict(name="tiny_s64_d64", workload=workload(1, 1, 1, 64, 64, 64, 64),
                arch=arch_tiny(),
                searches=[objective(OBJ_ENERGY, 1, TILE_POW2, ORD_NORECOMP2,
                                    FUSE_FUSED | FUSE_SEPARATE)])


def config2():
    """BERT-base-shaped attention on the edge accelerator; energy, then latency."""
    return dict(name="bert_base_s512", workload=workload(1, 12, 12, 512, 512, 64, 64),
                arch=arch_edge(),
                searches=[objective(OBJ_ENERGY, 1), objective(OBJ_LATENCY, 1)])


def config3():
    """Llama-style prefill attention on the cloud accelerator; energy and latency, top-16."""
    return dict(name="llama_prefill_s4096", workload=workload(1, 32, 32, 4096, 4096, 128, 128),
                arch=arch_cloud(),
                searches=[objective(OBJ_ENERGY, 16), objective(OBJ_LATENCY, 16)])


def config4():
    """Grouped-query attention (32 query heads on 8 KV heads), latency and energy-delay product."""
    return dict(name="gqa_b4_s8192", workload=workload(4, 32, 8, 8192, 8192, 128, 128),
                arch=arch_cloud(),
                searches=[objective(OBJ_LATENCY, 1), objective(OBJ_EDP, 1)])


SWEEP_SEQS = (1024, 2048, 4096, 8192, 16384, 32768, 65536)
SWEEP_HEAD_DIMS = (64, 128)


def config5():
    """Sweep: single-head attention at seq 1K..64K, d in {64,128}, edge and cloud, energy."""
    points = []
    for arch_name, mk in (("edge", arch_edge), ("cloud", arch_cloud)):
        for d in SWEEP_HEAD_DIMS:
            for s in SWEEP_SEQS:
                points.append(dict(name="sweep_%s_d%d_s%d" % (arch_name, d, s),
                                   workload=workload(1, 1, 1, s, s, d, d), arch=mk(),
                                   searches=[objective(OBJ_ENERGY, 1)]))
    return points


def all_configs():
    return [config1(), config2(), config3(), config4()] + config5()


# --- beyond attention: two GEMMs and convolution chains (Section VII-J), buffer-size sweeps ------

def two_gemm(I, K, L, J, word_bytes=2):
    """C = A(I x K) * B(K x L), E = C * D(L x J) as a single-instance workload."""
    return workload(1, 1, 1, I, L, K, J, word_bytes)


def conv_chain(hw, c_in, c_mid, c_out, k1):
    """Two convolutions as GEMMs via im2col: a k1 x k1 convolution over hw pixels followed by a 1 x 1
    convolution.  I = pixels, K = c_in * k1^2, L = c_mid, J = c_out."""
    return two_gemm(hw, c_in * k1 * k1, c_mid, c_out)


def arch_dram_only(gb_bytes, pe=32):
    """Cost coefficients that make the energy key the DRAM traffic in words: the objective of the
    DRAM-access-versus-buffer-size studies (Section VII-C)."""
    return arch(pe, pe, 1, gb_bytes, 0, 1, 1.0, 0.0, 0.0, 0.0, c_softmax=0.0, energy_quantum_pj=1.0)


def beyond_attention_configs():
    """The four non-attention chains of the paper's applicability table, on its first accelerator."""
    shapes = [("mlp_768_64_384_64", two_gemm(768, 64, 384, 64)),
              ("ffn_2048_768_3072_768", two_gemm(2048, 768, 3072, 768)),
              ("conv_chain_cc1", conv_chain(112 * 112, 64, 192, 128, 3)),
              ("conv_chain_cc2", conv_chain(56 * 56, 64, 64, 64, 1))]
    return [dict(name=n, workload=w, arch=arch_accel1(),
                 searches=[objective(OBJ_ENERGY, 1, fuse_mask=FUSE_FUSED)]) for n, w in shapes]


FFN_SWEEP_BUFFER_BYTES = tuple(64 * KiB << i for i in range(0, 10))      # 64 KB .. 32 MB


def ffn_dram_sweep_configs():
    """Fused feed-forward GEMMs of GPT-3-6.7B (32k x 4k x 16k and 32k x 16k x 4k, Section VII-C):
    the least DRAM traffic at each buffer size; 40 560 tilings x 18 750 rows x 9 mappings each."""
    w = two_gemm(32768, 4096, 16384, 4096)
    return [dict(name="ffn_gpt3_dram_%dKB" % (b // KiB), workload=w, arch=arch_dram_only(b),
                 searches=[objective(OBJ_ENERGY, 1, fuse_mask=FUSE_FUSED)]) for b in FFN_SWEEP_BUFFER_BYTES]


SM_WS_WS, SM_ALL = 0x001, 0x1ff      # stationary-pair masks: weight-stationary for both operators; all nine


def reconfigurable_array_designs(seq=512, d=64):
    """The four array designs of the paper's reconfigurable-array comparison (Section VII-K) for one
    BERT-Base-shaped head on its first accelerator, EDP-driven: fixed 32x32 weight-stationary array; free
    stationary modes on 32x32; free logical shape (every power-of-two rows x cols with 1024 PEs) under weight
    stationary; both.  Each entry: (name, stationary mask, list of (rows, cols))."""
    shapes = [(1 << a, 1024 >> a) for a in range(11)]
    cfg = dict(name="bert_base_s%d_accel1" % seq, workload=workload(1, 12, 12, seq, seq, d, d), arch=arch_accel1(),
               searches=[objective(OBJ_EDP, 1, fuse_mask=FUSE_FUSED)])
    designs = [("fixed_32x32_ws", SM_WS_WS, [(32, 32)]), ("ideal_flow_32x32", SM_ALL, [(32, 32)]),
               ("ideal_shape_ws", SM_WS_WS, shapes), ("ideal_shape_and_flow", SM_ALL, shapes)]
    return cfg, designs


def golden_configs():
    """Workloads whose exhaustive-search answers are stored under tests/golden/."""
    extra = [c for c in beyond_attention_configs() if c["name"] in ("mlp_768_64_384_64", "conv_chain_cc2")]
    sweep = [c for c in ffn_dram_sweep_configs() if c["name"] in ("ffn_gpt3_dram_1024KB",)]
    return all_configs() + extra + sweep


# --- seeded tiny problems for exhaustive parity ----------------------------------------------

def random_tiny_problem(seed: int):
    """A small random attention shape with a random accelerator, fully determined by `seed`.
    Dimensions are products of small primes so that divisor lists are ragged; capacities are
    chosen so that some, but not all, candidates fit."""
    rng = random.Random(seed)
    pick = lambda xs: xs[rng.randrange(len(xs))]
    seq_q = pick([4, 6, 8, 9, 12, 16, 18, 24])
    seq_kv = pick([4, 6, 8, 10, 12, 16, 20])
    d_qk = pick([2, 3, 4, 6, 8])
    d_v = pick([2, 4, 5, 6, 8])
    g = pick([1, 1, 2])
    kv = pick([1, 2])
    w = workload(pick([1, 2]), g * kv, kv, seq_q, seq_kv, d_qk, d_v, pick([1, 2, 4]))
    pe = pick([2, 4, 8])
    gb_words = pick([24, 48, 96, 200, 400, 1000])
    quantum = pick([1.0, 0.5, 0.25])
    a = arch(pe, pick([2, 4, 8]), pick([1, 2, 4]), gb_words * w["word_bytes"],
             pick([0, 64]), pick([1, 2, 3, 8]),
             quantum * rng.randrange(50, 400), quantum * rng.randrange(2, 20),
             quantum * rng.randrange(1, 4), quantum * rng.randrange(1, 4),
             c_softmax=float(rng.randrange(1, 12)), energy_quantum_pj=quantum)
    o = objective(pick([OBJ_ENERGY, OBJ_LATENCY, OBJ_EDP]), pick([1, 3, 16]),
                  pick([TILE_POW2, TILE_ALL_DIVISORS]), pick([ORD_NORECOMP2, ORD_ALL6]),
                  pick([1, 5, 7, 7, 3, 6]))
    return dict(name="tiny_seed%d" % seed, workload=w, arch=a, searches=[o])
