"""Hand-worked pins for the parts of the oracle that no printed number reaches: the serving memory and time model,
the training communication terms and the composition of the step time, and the analytic pipeline closed forms.

Every expected value below is a literal worked out on paper in the test's docstring, on models whose sizes are
powers of two and clusters whose rates are powers of two, so that each term is a short dyadic fraction (times are
quoted in units of u = 2^-20 s).  The regimes are chosen so that a term reduces to its textbook meaning: a
memory-bound decode step is bytes / HBM rate, a compute-bound prefill chunk is FLOPs / (peak x efficiency), a ring
all-reduce moves 2(n-1)/n of the buffer, an all-to-all (n-1)/n.  No GPU."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
from oracle import Oracle
from workloads import make_config

from helpers import axis_index, load_rows

U = 2.0 ** -20  # the time unit of the docstrings


# ----------------------------------------------------------------------------- serving

def hand_serve(mla: bool = False) -> dict:
    """Two layers, hidden 1024, 8 heads of 128, 8 experts of width 512, top-2, vocabulary 1000; 2 GPUs with
    peak 2^50 FLOP/s, HBM 2^40 B/s, link 2^30 B/s + 2^-20 s; every efficiency 0.5; requests (4096, 512) and
    (1024, 512)."""
    cfg = make_config("serve")
    cfg["model"].update(L=2, H=1024, nh=8, nkv=8, hd=128, attn_kind=1 if mla else 0,
                        kv_latent=512 if mla else 0, rope_dim=64 if mla else 0, E=8, K=2, F=512, S=0, Fs=0,
                        seq=0, vocab=1000)
    cfg["cluster"].update(G=8, budget_bytes=10 ** 15, peak_flops=float(2 ** 50), hbm_bw=float(2 ** 40),
                          bw_intra=float(2 ** 30), bw_inter=float(2 ** 30), alpha_intra=2.0 ** -20,
                          alpha_inter=2.0 ** -20)
    cfg["workload"].update(world=2, scen_P=[4096, 1024], scen_O=[512, 512])
    for k in cfg["kern"]:
        k["avail_mask"] = 255
        k["eff"] = [0.5] * 8
    cfg["axes"] = [("kv", [0, 3]), ("chunk", [1024, 4096]), ("batch", [1, 2]), ("dpa", [0, 1]), ("ep", [1, 2]),
                   ("tp", [1, 2]), ("scen", [0, 1])]
    return cfg


def test_serving_memory_hand_computed_mha():
    """tp = ep = 1, one request in flight, prompt 4096 + output 512, prefill chunk 4096, bf16 experts.
      attention 4 x 1024 x 1024 = 4,194,304 params; router 1024 x 8 = 8,192; one expert 3 x 1024 x 512 = 1,572,864
      weights: 2 layers x 2 B x (4,194,304 + 8,192 + 8 x 1,572,864) = 67,141,632, embedding + head 2 x 2 B x
        1,024,000 = 4,096,000                                                       -> 71,237,632
      KV bytes per token per layer: K and V, 8 heads x 128, bf16 = 4,096
      KV cache: 1 request x (4096 + 512) tokens x 2 layers x 4,096                  -> 37,748,736
      prefill workspace 8 x 2 B x 4096 x 1024                                       -> 67,108,864
      total 176,095,232 B."""
    cfg = hand_serve()
    d = Oracle(cfg).eval(axis_index(cfg, kv=0, chunk=4096, batch=1, dpa=0, ep=1, tp=1, scen=0))
    assert d["reason"] & 0x7F == 0
    assert d["bytes_w"] == 71_237_632
    assert d["bytes_a"] == 67_108_864
    assert d["mem"] == 71_237_632 + 37_748_736 + 67_108_864 == 176_095_232
    # two experts ranks (dp-attention, ep = 2, two requests in flight = one per rank): half the experts per GPU
    #   weights 2 x 2 x (4,194,304 + 8,192 + 4 x 1,572,864) + 4,096,000 = 46,071,808; cache of ONE request
    d = Oracle(cfg).eval(axis_index(cfg, kv=0, chunk=4096, batch=2, dpa=1, ep=2, tp=1, scen=0))
    assert d["reason"] & 0x7F == 0
    assert d["bytes_w"] == 46_071_808
    assert d["mem"] == 46_071_808 + 37_748_736 + 67_108_864 == 150_929_408


def test_serving_memory_hand_computed_mla_latent_is_not_sharded_by_tp():
    """Latent attention (latent 512 + rope 64), tp = 2 without dp-attention, two requests of 1024 + 512 tokens,
    prefill chunk 1024.
      attention: q 1024 x 8 x 128 + down-projection 1024 x 576 + up-projection 512 x 8 x 2 x 128 + o 8 x 128 x 1024
        = 1,048,576 + 589,824 + 1,048,576 + 1,048,576 = 3,735,552 params, half per GPU
      weights: 2 layers x (1,867,776 x 2 B + 8,192 x 2 B + 8 experts x 786,432 x 2 B) + 2 x 512,000 x 2 B
        = 2 x 16,334,848 + 2,048,000 = 34,717,696
      KV bytes per token per layer: (512 + 64) x 2 B = 1,152 on EVERY tensor-parallel rank (the latent is replicated;
        dividing it by tp would give 576)
      cache: 2 requests x 1,536 tokens x 2 layers x 1,152 = 7,077,888; workspace 8 x 2 x 1024 x 1024 = 16,777,216
      total 58,572,800 B.  With the fp8 variant the expert weights take 1 B each: 12,582,912 less -> 45,989,888."""
    cfg = hand_serve(mla=True)
    o = Oracle(cfg)
    d = o.eval(axis_index(cfg, kv=0, chunk=1024, batch=2, dpa=0, ep=1, tp=2, scen=1))
    assert d["reason"] & 0x7F == 0
    assert d["bytes_w"] == 34_717_696 and d["mem"] == 58_572_800
    d8 = o.eval(axis_index(cfg, kv=3, chunk=1024, batch=2, dpa=0, ep=1, tp=2, scen=1))
    assert d8["reason"] & 0x7F == 0
    assert d8["bytes_w"] == 22_134_784 and d8["mem"] == 45_989_888
    assert o.derived()["P_attn"] == 3_735_552 and o.derived()["dk"] == 576


def test_serving_time_memory_bound_decode_and_compute_bound_prefill():
    """tp = ep = 1, one request, prompt 4096, output 512, chunk 4096 (u = 2^-20 s).
    Decode step at the mean context 4096 + 512/2 = 4352 tokens: every layer streams its attention weights
    (8,388,608 B), the request's KV cache (4352 x 4,096 = 17,825,792 B) and the two experts the token routes to
    (2 x 3,145,728 B): 32,505,856 B = 31 x 2^20 B at 2^40 B/s = 31 u per layer; the FLOPs of one token at 2^49
    effective FLOP/s are thousands of times shorter.  T_dec = 2 layers x 31 u = 62 u.
    Prefill, one chunk of 4096 tokens: attention 4096 x (2 x 4,194,304 + 4 x 2048 x 8 x 128) = 2^36 FLOPs at 2^49 =
    2^-13 s; experts 4096 x 2 x 2 x 1,572,864 = 6 x 2^32 FLOPs at 2^49 = 6 x 2^-17 s (streaming all eight experts
    would take 24 u = 3 x 2^-17 s: compute-bound).  T_pre = 2 layers x (16 + 6) x 2^-17 s = 44 x 2^-17 s = 352 u.
    Throughput: 512 tokens / (352 u + 512 x 62 u) = 512 x 2^20 / 32,096 = 16,727.0349 tokens/s/GPU."""
    cfg = hand_serve()
    d = Oracle(cfg).eval(axis_index(cfg, kv=0, chunk=4096, batch=1, dpa=0, ep=1, tp=1, scen=0))
    assert d["reason"] & 0x7F == 0
    assert d["T_dec"] == pytest.approx(62 * U, rel=1e-13)
    assert d["T_pre"] == pytest.approx(352 * U, rel=1e-13)
    assert d["tput"] == pytest.approx(512 * 2 ** 20 / 32096, rel=1e-13)
    assert d["tput"] == pytest.approx(16727.0349, rel=1e-8)
    # the same prompt in four chunks of 1024 tokens: per chunk and layer, attention 1024 x 2^24 FLOPs at 2^49 =
    # 2^-15 s = 32 u (its weights stream in 8 u), experts 1024 x 6 x 2^20 FLOPs = 3 u of compute but all eight
    # experts stream in 24 u: memory-bound.  T_pre = 4 chunks x 2 layers x (32 + 24) u = 448 u.
    d4 = Oracle(cfg).eval(axis_index(cfg, kv=0, chunk=1024, batch=1, dpa=0, ep=1, tp=1, scen=0))
    assert d4["T_pre"] == pytest.approx(448 * U, rel=1e-13) and d4["T_dec"] == d["T_dec"]


def test_serving_dp_attention_all_to_all_term():
    """dp-attention on two GPUs (tp = 1, ep = 2), two requests (one per rank), prompt 4096, output 512, chunk 4096.
    Per layer and decode step each rank sends its token's 2 routed copies of 1024 bf16 values = 4,096 B; an
    all-to-all over 2 ranks moves half of it: 2,048 B / 2^30 B/s = 2 u, plus 1 u latency, twice (dispatch and
    combine) = 6 u.  Attention streams 25 u as in the one-GPU case; the experts touched are min(4 local, 4 copies /
    2 ranks) = 2 -> 6 u.  T_dec = 2 x (25 + 6 + 6) u = 74 u.
    Prefill chunk: the all-to-all carries 2 B x 4096 x 2 x 1024 = 2^24 B, half of it at 2^30 B/s = 2^-7 s, + 1 u, twice
    = 16,384 u + 2 u; attention 2^-13 s = 128 u; experts 6 x 2^32 FLOPs over two GPUs = 3 x 2^-17 s = 24 u (four
    local experts stream in 12 u).  T_pre = 2 x (128 + 24 + 16,386) u = 33,076 u.
    Throughput per GPU: 2 x 512 tokens / (33,076 u + 512 x 74 u) / 2 GPUs = 512 x 2^20 / 70,964 = 7,565.3981."""
    cfg = hand_serve()
    d = Oracle(cfg).eval(axis_index(cfg, kv=0, chunk=4096, batch=2, dpa=1, ep=2, tp=1, scen=0))
    assert d["reason"] & 0x7F == 0
    assert d["T_dec"] == pytest.approx(74 * U, rel=1e-13)
    assert d["T_pre"] == pytest.approx(33076 * U, rel=1e-13)
    assert d["tput"] == pytest.approx(512 * 2 ** 20 / 70964, rel=1e-13)


def test_serving_tensor_parallel_all_reduce_term():
    """tp = 2 without dp-attention, two requests, prompt 1024, output 512, chunk 1024.  Per layer and decode step the
    two activations of 1024 bf16 values (4,096 B) are all-reduced twice: a ring over 2 ranks moves 2 x 1/2 x 4,096 B
    at 2^30 B/s = 2^-18 s = 4 u, plus 2 x 1 hop x 1 u latency = 6 u; twice: 12 u.
    Attention: half the weights (4,194,304 B) + 2 requests x 1280 context tokens x 2,048 B (K/V heads split over tp)
    = 9,437,184 B = 9 u; experts: min(8, 4 copies) = 4 experts x 3,145,728 B / 2 (expert matrices split over tp) =
    6 u.  T_dec = 2 x (9 + 6 + 12) u = 54 u."""
    cfg = hand_serve()
    d = Oracle(cfg).eval(axis_index(cfg, kv=0, chunk=1024, batch=2, dpa=0, ep=1, tp=2, scen=1))
    assert d["reason"] & 0x7F == 0
    assert d["T_dec"] == pytest.approx(54 * U, rel=1e-13)


# ----------------------------------------------------------------------------- training on 8 GPUs

def hand_train(G: int = 8) -> dict:
    """Four layers, hidden 1024, 8 heads of 128, 4 experts of width 512, top-2, sequence 1024, vocabulary 1024,
    embeddings not counted; 16 sequences per step, microbatch 1; peak 2^40 FLOP/s, HBM 2^40 B/s, intra-node link
    2^30 B/s + 2^-20 s, inter-node 2^28 B/s + 2^-18 s; every efficiency 0.5, backward = 2 x forward, half of the
    gradient reduction hidden.  Schedules: 0 = 1F1B, 1 = interleaved with overlap (half of the all-to-all hidden,
    25 % schedule overhead), 2 = DualPipe-style (mapped here, no overlap).  Kernel 1 pays a 25 % patch overhead."""
    cfg = make_config("tiny")
    cfg["model"].update(L=4, H=1024, nh=8, nkv=8, hd=128, E=4, K=2, F=512, S=0, Fs=0, seq=1024, vocab=1024,
                        count_embeddings=0)
    cfg["cluster"].update(G=G, budget_bytes=10 ** 15, peak_flops=float(2 ** 40), hbm_bw=float(2 ** 40),
                          bw_intra=float(2 ** 30), bw_inter=float(2 ** 28), alpha_intra=2.0 ** -20,
                          alpha_inter=2.0 ** -18)
    cfg["workload"].update(gbs=16, world=8)
    cfg["rules"].update(world_min=1, world_max=64, ep_scope=0)
    for k in cfg["kern"]:
        k["avail_mask"] = 255
        k["eff"] = [0.5] * 8
    cfg["kern"][1]["patch_ovh"] = 0.25
    cfg["sched"][1].update(overlap=1, hide_frac=0.5, sched_ovh=0.25)
    cfg["sched"][2].update(mapped=1, overlap=0, hide_frac=0.0)
    cfg["axes"] = [("kv", [0, 1]), ("rec", [0, 1, 2]), ("sched", [0, 1, 2]), ("mb", [1]), ("v", [0]),
                   ("ep", [1, 2]), ("pp", [1, 2]), ("tp", [1, 2]), ("dp", [1, 2]), ("world", [0])]
    return cfg


def test_training_step_time_hand_computed_tp2_pp2_ep2_dp2():
    """1F1B, no recompute, tp = pp = ep = dp = 2 on one 8-GPU node; m = 16 / (2 x 1) = 8 microbatches of t = 1024
    tokens; two layers per stage.  Times in u = 2^-20 s.
      dense FLOPs/token/layer: attention 2 x 4,194,304 + 2 x 1024 x 8 x 128 = 10 x 2^20, router 2 x 1024 x 4 = 2^13;
        over tp = 2 at 2^39 effective FLOP/s: 1024 x (10 x 2^20 + 2^13) / 2^40 s = 10,240 u + 8 u
      expert FLOPs/token/layer: 2 x 2 x 1,572,864 = 6 x 2^20 -> 6,144 u             cF = 16,392 u,  cB = 32,784 u
      tokens per expert 1024 x 2 x 2 / 4 = 1024 (bucket 4)
      TP all-reduce of 2 B x 1024 x 1024 = 2^21 B over 2 ranks: ring 2 x 1/2 x 2^21 / 2^30 s = 2,048 u + 2 x 1 hop x
        1 u = 2,050 u, twice per layer pass                                          tpc = 4,100 u
      EP all-to-all of 2 B x 1024 x 2 x 1024 / tp = 2^21 B over 2 ranks: 1/2 x 2^21 / 2^30 s = 1,024 u + 1 u, twice
                                                                                     a2a = 2,050 u
      F_l = 16,392 + 4,100 + 2,050 = 22,542 u;  B_l = 32,784 + 4,100 + 2,050 = 38,934 u
      head: 1024 x 2 x 1024 x 1024 / 2^40 s = 2,048 u forward, amortised over the two stages
      F = 2 x 22,542 + 1,024 = 46,108 u;  B = 2 x 38,934 + 2,048 = 79,916 u
      stage hand-over: 2^21 B / tp at 2^30 B/s + 1 u = 1,025 u
      T_pipe = (8 + 2 - 1) x 126,024 + 2 x 1 x 1,025 = 1,136,266 u
      parameters per GPU: dense 2 x (2,097,152 + 4,096) = 4,202,496; experts 2 layers x 2 experts x 786,432 = 3,145,728
      gradient reduce-scatter + weight all-gather over dp = 2 of 6 B x 4,202,496 = 25,214,976 B: 2 x 1/2 x that /
        2^30 s = 24,624 u + 2 u; the experts' group has one member                   T_dp = 24,626 u
      optimizer state 12 B x (2,101,248 + 3,145,728) = 62,963,712 B, read and written once: 120.09375 u
      T_step = 1,136,266 + 24,626 / 2 + 120.09375 = 1,148,699.09375 u
      throughput = 16 x 1024 tokens / (T_step x 8 GPUs) = 2048 x 2^20 / 1,148,699.09375 = 1,869.4919 tokens/s/GPU."""
    cfg = hand_train()
    o = Oracle(cfg)
    d = o.eval(axis_index(cfg, kv=0, rec=0, sched=0, ep=2, pp=2, tp=2, dp=2))
    assert d["reason"] == 0 and d["world"] == 8 and d["m"] == 8 and d["m_e"] == 1024 and d["bucket"] == 4
    assert (d["N_dense"], d["N_exp"], d["bytes_o"]) == (4_202_496, 3_145_728, 62_963_712)
    want = dict(cF=16392, cB=32784, tpc=4100, a2a=2050, F_l=22542, B_l=38934, headF=2048, F=46108, B=79916, p=1025,
                T_pipe=1136266, T_dp=24626, T_opt=120.09375, T_step=1148699.09375)
    for name, units in want.items():
        assert d[name] == pytest.approx(units * U, rel=1e-13), name
    assert d["tput"] == pytest.approx(2048 * 2 ** 20 / 1148699.09375, rel=1e-13)
    assert d["tput"] == pytest.approx(1869.4919, rel=1e-8)
    # the non-native kernel variant pays its 25 % patch overhead on the same plan
    d1 = o.eval(axis_index(cfg, kv=1, rec=0, sched=0, ep=2, pp=2, tp=2, dp=2))
    assert d1["tput"] == pytest.approx(d["tput"] / 1.25, rel=1e-13)


def test_training_links_switch_to_the_inter_node_rates_beyond_a_node():
    """The same plan on nodes of 2 GPUs: tensor parallelism (2 ranks) stays inside a node, the expert group spans
    tp x ep = 4 GPUs, the data-parallel group tp x dp = 4 and the pipeline the whole world, so those three use
    2^28 B/s + 4 u:
      all-to-all 2 x (1/2 x 2^21 / 2^28 s + 4 u) = 2 x (4,096 + 4) = 8,200 u;  hand-over 2^20 / 2^28 s + 4 u = 4,100 u
      gradient exchange 25,214,976 B / 2^28 s = 98,496 u + 2 x 4 u = 98,504 u;  TP all-reduce unchanged 4,100 u."""
    cfg = hand_train(G=2)
    d = Oracle(cfg).eval(axis_index(cfg, kv=0, rec=0, sched=0, ep=2, pp=2, tp=2, dp=2))
    assert d["reason"] == 0
    for name, units in dict(tpc=4100, a2a=8200, p=4100, T_dp=98504).items():
        assert d[name] == pytest.approx(units * U, rel=1e-13), name


def test_training_overlap_hides_part_of_the_all_to_all_and_is_priced():
    """Interleaved schedule with overlap on the same layout (two virtual stages of one layer per rank): half of the
    2,050 u all-to-all hides behind the layer's compute (which is far longer), in both passes:
      F_l = 16,392 + 4,100 + 1,025 = 21,517 u;  B_l = 32,784 + 4,100 + 1,025 = 37,909 u
      F = 2 x 21,517 + 1,024 = 44,058 u;  B = 2 x 37,909 + 2,048 = 77,866 u
      T_pipe = (8 + (2 - 1)/2) x 121,924 + 2 x (4 - 1) x 1,025 = 1,036,354 + 6,150 = 1,042,504 u
      T_step = 1,042,504 + 12,313 + 120.09375 = 1,054,937.09375 u;  the score is divided by 1 + 0.25."""
    cfg = hand_train()
    d = Oracle(cfg).eval(axis_index(cfg, kv=0, rec=0, sched=1, ep=2, pp=2, tp=2, dp=2))
    assert d["reason"] == 0 and d["v_eff"] == 2 and d["Q"] == 4
    for name, units in dict(xF=1025, xB=1025, F_l=21517, B_l=37909, F=44058, B=77866, T_pipe=1042504,
                            T_step=1054937.09375).items():
        assert d[name] == pytest.approx(units * U, rel=1e-13), name
    assert d["tput"] == pytest.approx(2048 * 2 ** 20 / 1054937.09375 / 1.25, rel=1e-13)


def test_hidden_all_to_all_is_capped_by_the_compute_it_hides_behind():
    """The same interleaved + overlap plan behind a link of 2^20 B/s: the all-to-all takes 2 x (1/2 x 2^21 B / 2^20 B/s
    + 1 u) = 2,097,154 u, far longer than a layer's compute, so it can hide only behind what compute there is: the
    forward's 16,392 u, and in the backward pass 32,784 u plus the 4,096 u that selective recompute re-runs.
      xF = 2,097,154 - 16,392 = 2,080,762 u;  xB = 2,097,154 - 36,880 = 2,060,274 u."""
    cfg = hand_train()
    cfg["cluster"].update(bw_intra=float(2 ** 20))
    d = Oracle(cfg).eval(axis_index(cfg, kv=0, rec=1, sched=1, ep=2, pp=2, tp=2, dp=2))
    assert d["reason"] == 0
    for name, units in dict(a2a=2097154, cF=16392, cB=32784, rc=4096, xF=2080762, xB=2060274).items():
        assert d[name] == pytest.approx(units * U, rel=1e-12), name


def test_training_dualpipe_style_closed_form_and_second_stage_copy():
    """DualPipe-style class on the same layout: every rank holds two stage copies, so its parameters double
    (dense 8,404,992, experts 6,291,456; optimizer state 125,927,424 B -> 240.1875 u), the gradient exchange too
    (50,429,952 B / 2^30 s = 49,248 u + 2 u), and
      T_pipe = 8 x 126,024 + max(2 - 2, 0) x B + 126,024 / 8 + 2 x 1,025 = 1,008,192 + 15,753 + 2,050 = 1,025,995 u
      T_step = 1,025,995 + 24,625 + 240.1875 = 1,050,860.1875 u."""
    cfg = hand_train()
    d = Oracle(cfg).eval(axis_index(cfg, kv=0, rec=0, sched=2, ep=2, pp=2, tp=2, dp=2))
    assert d["reason"] == 0
    assert (d["N_dense"], d["N_exp"], d["bytes_o"]) == (8_404_992, 6_291_456, 125_927_424)
    for name, units in dict(T_pipe=1025995, T_dp=49250, T_opt=240.1875, T_step=1050860.1875).items():
        assert d[name] == pytest.approx(units * U, rel=1e-13), name


def test_recompute_terms_hand_computed():
    """Recompute on the 1F1B plan above.  Selective re-runs the expert FFN in the backward pass: two of its three
    GEMMs' worth, 2/3 x 6,144 u = 4,096 u (no shared experts here); full re-runs the whole forward, 16,392 u of compute
    plus the forward's collectives (4,100 + 2,050 u) once more:
      selective B_l = 38,934 + 4,096 = 43,030 u;  full B_l = 38,934 + 16,392 + 6,150 = 61,476 u."""
    cfg = hand_train()
    o = Oracle(cfg)
    sel = o.eval(axis_index(cfg, kv=0, rec=1, sched=0, ep=2, pp=2, tp=2, dp=2))
    full = o.eval(axis_index(cfg, kv=0, rec=2, sched=0, ep=2, pp=2, tp=2, dp=2))
    assert sel["reason"] == 0 and full["reason"] == 0
    assert sel["rc"] == pytest.approx(4096 * U, rel=1e-12) and sel["B_l"] == pytest.approx(43030 * U, rel=1e-12)
    assert full["rc"] == pytest.approx(16392 * U, rel=1e-13) and full["B_l"] == pytest.approx(61476 * U, rel=1e-13)
    assert sel["F_l"] == full["F_l"] == pytest.approx(22542 * U, rel=1e-13)


# ----------------------------------------------------------------------------- closed forms vs the event simulation

def _uniform_pipeline_cfg():
    """A space with uniform stages and free stage hand-overs: no head (vocabulary 0), layers divisible by every
    pp x v used, zero latency and an (in fp32) infinite link."""
    cfg = hand_train()
    cfg["model"].update(L=16, vocab=0)
    big = float(np.float32(1e30))
    cfg["cluster"].update(bw_intra=big, bw_inter=big, alpha_intra=0.0, alpha_inter=0.0)
    cfg["workload"].update(gbs=64)
    cfg["sched"][1].update(overlap=0, hide_frac=0.0, sched_ovh=0.0)
    cfg["axes"] = [("kv", [0]), ("rec", [0]), ("sched", [0, 1, 2]), ("mb", [1, 2]), ("v", [1, 2, 4]),
                   ("ep", [1]), ("pp", [1, 2, 4, 8]), ("tp", [1]), ("dp", [1, 2]), ("world", [0])]
    return cfg


def test_analytic_pipeline_time_equals_event_simulation_for_uniform_stages():
    """With uniform stages, free hand-overs and no jitter the 1F1B closed form (m + pp - 1)(F + B) and the
    interleaved one (m + (pp - 1)/v)(F + B) are what the event-driven evaluation of the same schedule orders
    gives: the analytic tier and the simulator tier agree where they must."""
    cfg = _uniform_pipeline_cfg()
    o = Oracle(cfg)
    n1 = ni = 0
    for i in range(o.size):
        d = o.eval(i)
        if d["reason"] & 0x7F or d["kind"] == 2:
            continue
        pp, v, m = d["pp"], d["v_eff"], d["m"]
        Q = pp * v
        assert d["p"] < 1e-20
        Fq, Bq = [d["F"] / v] * Q, [d["B"] / v] * Q
        got = oracle.makespan(d["kind"], pp, v, m, Fq, Bq, 0.0)
        assert got == pytest.approx(d["T_pipe"], rel=1e-12), (pp, v, m, d["kind"])
        n1 += d["kind"] == 0
        ni += d["kind"] == 1
    assert n1 >= 8 and ni >= 8


def test_dualpipe_style_closed_form_against_event_simulation():
    """The DualPipe-style analytic form is m (F + B) + max(pp - 2, 0) B + (F + B) / startup_div.  Its first two terms
    are checked against event-simulated makespans of the DualPipe-style order (F = 1, B = 2, free hand-overs; the
    golden file comes from an implementation that is not the oracle's): they never exceed the simulated makespan, stay
    within pp ticks of it, and equal it in eight of the twelve tabulated shapes (the order's greedy choices cost a few
    ticks in the other four); the startup term is this repo's reading of the printed divisor (8.0) and is what the
    analytic tier adds on top."""
    cfg = _uniform_pipeline_cfg()
    cfg["axes"][2] = ("sched", [2])
    cfg["axes"][6] = ("pp", [1, 2, 4, 8, 16])
    cfg["axes"][3] = ("mb", [1])
    cfg["axes"][8] = ("dp", [1])
    golden = {(pp, m): t for f, b, pp, m, t in load_rows("dualpipe_style_makespans.txt") if (f, b) == (1, 2)}
    o = Oracle(cfg)
    exact = 0
    for gbs in (8, 16, 32, 64):
        cfg["workload"]["gbs"] = gbs
        o = Oracle(cfg)
        for i in range(o.size):
            d = o.eval(i)
            if d["reason"] & 0x7F or (d["pp"], d["m"]) not in golden:
                continue
            pp, m = d["pp"], d["m"]
            unit = d["F"]                       # B = 2 F with bwd_factor 2 and no head: the golden file's 1 : 2
            assert d["B"] == pytest.approx(2 * unit, rel=1e-12)
            body = d["T_pipe"] - (d["F"] + d["B"]) / 8.0
            assert body == pytest.approx((3 * m + 2 * max(pp - 2, 0)) * unit, rel=1e-12)
            sim = golden[(pp, m)] * unit
            assert body <= sim * (1 + 1e-12)
            assert sim <= body + pp * unit * (1 + 1e-12)
            if (pp, m) in ((4, 8), (4, 16), (4, 32), (4, 64), (8, 8), (8, 32), (8, 64), (16, 16)):
                assert body == pytest.approx(sim, rel=1e-12), (pp, m)
                exact += 1
    assert exact == 8


def test_golden_files_regenerate_from_their_committed_script():
    """The two golden files without a printed source are reproducible: the script beside them (numpy predicates for
    the rule counts, a pure-Python event simulation for the DualPipe-style makespans; it imports neither the oracle
    nor the CUDA package) gives the stored values."""
    import os
    import subprocess
    import sys
    from helpers import GOLDEN
    src = open(os.path.join(GOLDEN, "make_goldens.py")).read()
    assert "import oracle" not in src and "from oracle" not in src and "paper_2607_18631_b200" not in src
    r = subprocess.run([sys.executable, os.path.join(GOLDEN, "make_goldens.py"), "--check"], capture_output=True,
                       text=True)
    assert r.returncode == 0, r.stdout + r.stderr


# ----------------------------------------------------------------------------- serving with leading dense layers

def hand_serve_dense() -> dict:
    """hand_serve() with three layers of which the first carries a plain FFN of width 2048 instead of experts:
    attention 4,194,304 + FFN 3 x 1024 x 2048 = 10,485,760 parameters, 20 x 2^20 bytes in bf16."""
    cfg = hand_serve()
    cfg["model"].update(L=3, L_dense=1, F_dense=2048)
    return cfg


def test_serving_leading_dense_layer_hand_computed():
    """tp = ep = 1, one request, prompt 4096, output 512, chunk 4096 (u = 2^-20 s).
    Memory: two MoE layers 2 x 33,570,816 B + the dense layer 20,971,520 B + embedding and head 4,096,000 B =
    92,209,152 B of weights; KV cache 4608 tokens x 3 layers x 4,096 B = 56,623,104; workspace 67,108,864;
    total 215,941,120 B.
    Decode: a MoE layer streams 31 u as before; the dense layer streams its 20 x 2^20 B of weights and the 17 x 2^20 B
    of KV cache: 37 u.  T_dec = 2 x 31 + 37 = 99 u.
    Prefill: a MoE layer 176 u as before; the dense layer 4096 x (2 x 10,485,760 + 4 x 2048 x 8 x 128) = 28 x 2^32
    FLOPs at 2^49 = 224 u (its weights stream in 20 u: compute-bound).  T_pre = 2 x 176 + 224 = 576 u.
    Throughput 512 x 2^20 / (576 + 512 x 99) = 512 x 2^20 / 51,264."""
    cfg = hand_serve_dense()
    d = Oracle(cfg).eval(axis_index(cfg, kv=0, chunk=4096, batch=1, dpa=0, ep=1, tp=1, scen=0))
    assert d["reason"] & 0x7F == 0
    assert d["bytes_w"] == 92_209_152 and d["mem"] == 215_941_120
    assert d["T_dec"] == pytest.approx(99 * U, rel=1e-13)
    assert d["T_pre"] == pytest.approx(576 * U, rel=1e-13)
    assert d["tput"] == pytest.approx(512 * 2 ** 20 / 51264, rel=1e-13)


def test_serving_leading_dense_layer_is_sharded_and_all_reduced_over_tp():
    """tp = 2 without dp-attention, two requests, prompt 1024, output 512, chunk 1024.  The dense layer's weights
    halve (10 u), its KV reads are those of the MoE layers (2 x 1280 x 2,048 B = 5 u), and its two all-reduces of
    the two requests' activations cost 2 x (4 u + 2 u) = 12 u like a MoE layer's: 27 u.  T_dec = 2 x 27 + 27 = 81 u.
    Weights per GPU: 2 x (4,194,304 + 16,384 + 8 x 1,572,864) + 10,485,760 + 2,048,000 = 33,587,200 + 12,533,760 =
    46,120,960 B."""
    cfg = hand_serve_dense()
    d = Oracle(cfg).eval(axis_index(cfg, kv=0, chunk=1024, batch=2, dpa=0, ep=1, tp=2, scen=1))
    assert d["reason"] & 0x7F == 0
    assert d["bytes_w"] == 46_120_960
    assert d["T_dec"] == pytest.approx(81 * U, rel=1e-13)


def test_serving_without_dense_layers_is_unchanged_by_the_dense_fields():
    """L_dense = 0: the width of a dense FFN that no layer has changes nothing, to the bit."""
    a, b = hand_serve(), hand_serve()
    b["model"].update(F_dense=4096)
    ra, ta, ma, _ = Oracle(a).score_range()
    rb, tb, mb, _ = Oracle(b).score_range()
    np.testing.assert_array_equal(ra, rb)
    np.testing.assert_array_equal(ta, tb)
    np.testing.assert_array_equal(ma, mb)


# ----------------------------------------------------------------------------- the sharding regimes, by hand

def hand_train_sharded() -> dict:
    """hand_train() with the sharding axis (0 zero1, 1 zero1 with the optimizer offloaded, 2 fully sharded), a host
    link of 2^26 B/s and a contention penalty of 25 %."""
    cfg = hand_train()
    cfg["axes"] = list(cfg["axes"]) + [("shard", [0, 1, 2])]
    cfg["cluster"]["bw_host"] = float(2 ** 26)
    cfg["consts"]["offload_overlap_penalty"] = 0.25
    return cfg


def test_offloaded_optimizer_step_time_hand_computed():
    """The plan of test_training_step_time_hand_computed_tp2_pp2_ep2_dp2 with the optimizer state in host memory.
    The rank owns the state of half its dense parameters (dp = 2) and of all its expert parameters (expert-DP group
    of one): 2,101,248 + 3,145,728 = 5,246,976 parameters.  Per step their fp32 gradients go down and their bf16
    weights come back over the host link: 6 B x 5,246,976 = 31,481,856 B at 2^26 B/s = 491,904 u, instead of
    120.09375 u of HBM sweeps.  Pipeline and gradient exchange are unchanged:
      T_step = 1,136,266 + 24,626 / 2 + 491,904 = 1,640,483 u;  throughput 2048 x 2^20 / 1,640,483.
    Memory: the 62,963,712 B of optimizer state leave the device, nothing else changes."""
    cfg = hand_train_sharded()
    o = Oracle(cfg)
    z = o.eval(axis_index(cfg, kv=0, rec=0, sched=0, ep=2, pp=2, tp=2, dp=2, shard=0))
    d = o.eval(axis_index(cfg, kv=0, rec=0, sched=0, ep=2, pp=2, tp=2, dp=2, shard=1))
    assert d["reason"] == 0 and z["reason"] == 0
    assert z["T_step"] == pytest.approx(1148699.09375 * U, rel=1e-13)          # zero1 = the plan without the axis
    assert d["T_opt"] == pytest.approx(491904 * U, rel=1e-13)
    assert d["T_dp"] == pytest.approx(24626 * U, rel=1e-13) and d["T_pipe"] == pytest.approx(1136266 * U, rel=1e-13)
    assert d["T_step"] == pytest.approx(1640483 * U, rel=1e-13)
    assert d["tput"] == pytest.approx(2048 * 2 ** 20 / 1640483, rel=1e-13)
    assert d["bytes_o"] == 0 and z["mem"] - d["mem"] == 62_963_712


def test_offload_switches_the_hiding_off_and_pays_the_contention_penalty_when_overlapped():
    """The interleaved + overlap plan of test_training_overlap_hides_part_of_the_all_to_all_and_is_priced (half of
    the 2,050 u all-to-all hidden under zero1, 25 % schedule overhead).  With the optimizer offloaded nothing is
    hidden (2,050 u exposed in both passes, so the layer times are those of the plan without overlap: 22,542 and
    38,934 u) and the plan pays the 25 % contention penalty on top of the schedule overhead:
      F = 2 x 22,542 + 1,024 = 46,108 u;  B = 2 x 38,934 + 2,048 = 79,916 u
      T_pipe = (8 + 1/2) x 126,024 + 6 x 1,025 = 1,071,204 + 6,150 = 1,077,354 u
      T_step = 1,077,354 + 12,313 + 491,904 = 1,581,571 u;  priced throughput = unpriced / (1.25 x 1.25)."""
    cfg = hand_train_sharded()
    o = Oracle(cfg)
    z = o.eval(axis_index(cfg, kv=0, rec=0, sched=1, ep=2, pp=2, tp=2, dp=2, shard=0))
    d = o.eval(axis_index(cfg, kv=0, rec=0, sched=1, ep=2, pp=2, tp=2, dp=2, shard=1))
    assert z["reason"] == 0 and d["reason"] == 0
    assert z["xF"] == pytest.approx(1025 * U, rel=1e-13) and z["xB"] == pytest.approx(1025 * U, rel=1e-13)
    assert z["tput"] == pytest.approx(2048 * 2 ** 20 / 1054937.09375 / 1.25, rel=1e-13)
    for name, units in dict(a2a=2050, xF=2050, xB=2050, F_l=22542, B_l=38934, F=46108, B=79916, T_pipe=1077354,
                            T_opt=491904, T_step=1581571).items():
        assert d[name] == pytest.approx(units * U, rel=1e-13), name
    assert d["tput_unpriced"] == pytest.approx(2048 * 2 ** 20 / 1581571, rel=1e-13)
    assert d["tput"] == pytest.approx(d["tput_unpriced"] / (1.25 * 1.25), rel=1e-13)
    # without overlap (1F1B) the offloaded plan pays neither overhead
    d0 = o.eval(axis_index(cfg, kv=0, rec=0, sched=0, ep=2, pp=2, tp=2, dp=2, shard=1))
    assert d0["tput"] == pytest.approx(d0["tput_unpriced"], rel=1e-13)


def test_fully_sharded_memory_and_exchange_hand_computed():
    """The same tp2 / pp2 / ep2 / dp2 plan, fully sharded.
    Memory: weights and gradients are held for the 5,246,976 parameters the rank owns: 2 B x 5,246,976 = 10,493,952
    and 4 B x 5,246,976 = 20,987,904 (replicated: 2 B and 4 B x 7,348,224 = 14,696,448 and 29,392,896); the
    optimizer state is unchanged (62,963,712); the all-gather buffer holds two layers of unsharded bf16 parameters:
    a layer is 2,097,152 (attention / tp) + 4,096 (router) + 2 local experts x 786,432 = 3,674,112 parameters ->
    2 x 2 B x 3,674,112 = 14,696,448 B.
    Exchange, per microbatch, over the dense data-parallel group of 2 (the expert group has one member and moves
    nothing): gather the bf16 dense weights for the forward and again for the backward, 1/2 x 2 B x 4,202,496 /
    2^30 s = 4,104 u + 1 u each; reduce-scatter the fp32 gradients, 1/2 x 4 B x 4,202,496 / 2^30 s = 8,208 u + 1 u:
    2 x 4,105 + 8,209 = 16,419 u, times 8 microbatches = 131,352 u (the replicated regimes exchange 24,626 u once).
      T_step = 1,136,266 + 131,352 / 2 + 120.09375 = 1,202,062.09375 u."""
    cfg = hand_train_sharded()
    o = Oracle(cfg)
    z = o.eval(axis_index(cfg, kv=0, rec=0, sched=0, ep=2, pp=2, tp=2, dp=2, shard=0))
    d = o.eval(axis_index(cfg, kv=0, rec=0, sched=0, ep=2, pp=2, tp=2, dp=2, shard=2))
    assert d["reason"] == 0
    assert (z["bytes_w"], z["bytes_g"], z["bytes_buf"]) == (14_696_448, 29_392_896, 0)
    assert (d["bytes_w"], d["bytes_g"], d["bytes_o"], d["bytes_buf"]) == (10_493_952, 20_987_904, 62_963_712, 14_696_448)
    assert d["mem"] - z["mem"] == (10_493_952 + 20_987_904 + 14_696_448) - (14_696_448 + 29_392_896)
    assert d["bytes_a"] == z["bytes_a"]
    assert d["T_dp"] == pytest.approx(131352 * U, rel=1e-13)
    assert d["T_opt"] == pytest.approx(120.09375 * U, rel=1e-13)
    assert d["T_step"] == pytest.approx(1202062.09375 * U, rel=1e-13)
    assert d["tput"] == pytest.approx(2048 * 2 ** 20 / 1202062.09375, rel=1e-13)


def test_activation_bytes_hand_computed_with_and_without_a_leading_dense_layer():
    """Activations kept per token and layer, bf16 (2 B) unless stated; hidden 1024, 8 + 8 + 8 heads of 128:
      attention: layer-norm input 1024 + projection input 1024 + q, k, v 3 x 1024 + output-projection input 1024
        = 6,144 values = 12,288 B
      MoE part kept under selective recompute: layer-norm input + router input 2 x 1024 values (4,096 B), fp32 router
        logits 4 x 4 B (16 B), two dispatched copies 2 x 1024 values (4,096 B), combine output 1024 values (2,048 B)
        = 10,256 B;  dropped by selective recompute: gate, up, act x up for two routed copies of width 512 =
        3 x 1,024 values = 6,144 B                          -> MoE layer: 28,688 B (none), 22,544 B (selective)
      leading dense layer of width 2048: layer-norm input + FFN input 4,096 B kept; gate, up, act x up 3 x 2048 values
        = 12,288 B dropped by selective recompute           -> dense layer: 28,672 B (none), 16,384 B (selective)
      full recompute keeps the layer input only: 2,048 B, and one layer is live while it is recomputed.
    Plan tp2 / pp2 / ep2 / dp2, 1F1B: 1024 tokens per microbatch, sharded over tp = 2 (sequence parallel), two layers
    per stage, min(pp, m) = 2 microbatches in flight on rank 0, whose first layer is the dense one:
      none       2 x (14,688,256 + 14,680,064) = 58,736,640    (two MoE layers: 2 x 2 x 14,688,256 = 58,753,024)
      selective  2 x (11,542,528 +  8,388,608) = 39,862,272
      full       2 x ( 1,048,576 +  1,048,576) + 14,688,256 = 18,882,560."""
    cfg = hand_train()
    plain = Oracle(cfg)
    cfg_d = hand_train()
    cfg_d["model"].update(L_dense=1, F_dense=2048)
    dense = Oracle(cfg_d)
    want = {0: (58_753_024, 58_736_640), 1: (2 * 2 * 11_542_528, 39_862_272),
            2: (2 * 2 * 1_048_576 + 14_688_256, 18_882_560)}
    for rec, (w_plain, w_dense) in want.items():
        i = axis_index(cfg, kv=0, rec=rec, sched=0, ep=2, pp=2, tp=2, dp=2)
        a, b = plain.eval(i), dense.eval(i)
        assert a["reason"] == 0 and b["reason"] == 0
        assert a["bytes_a"] == w_plain, rec
        assert b["bytes_a"] == w_dense, rec
    dv = dense.derived()
    assert (dv["a_attn"], dv["a_full"], dv["a_sel"], dv["a_ckpt"]) == (12_288, 28_688, 22_544, 2_048)
    assert (dv["a_full_d"], dv["a_sel_d"]) == (28_672, 16_384)
