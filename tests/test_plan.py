"""fa_plan: the host-side choice of kernel, tiling and split count (no GPU needed).

The expectations are the measured outcomes recorded for the B200 (148 SMs): the benchmark
configurations, the paper's Table 6 rows and the decode-like shapes."""
import pytest

from paper_2609_21264_b200 import binding, workloads as W

SMS = 148


def plan(w, **kw):
    return binding.fa_plan(SMS, w.B, w.Hq, w.Hkv, w.Sq, w.Sk, w.dqk, w.dv, w.causal, **kw)


def test_benchmark_configurations():
    # (config 3: 4096 items of up to 64 K/V tiles, 27 per SM: the persistent kernel; config 4: 4096 one-tile items of up
    #  to 32 K/V tiles at 192/128: the stream kernel's persistent form; config 5: items of 1024 tiles)
    expect = ["fa_fwd_stream", "fa_fwd_pair", "fa_fwd_persistent", "fa_fwd_stream_persistent", "fa_fwd_pair"]
    for w, kernel in zip(W.CONFIGS, expect):
        p = plan(w)
        assert p["kernel"] == kernel, (w.name, p)
        assert p["kv_splits"] == 1
    # grid sizes: one CTA per query tile or per pair of query tiles
    assert plan(W.CONFIGS[0])["ctas"] == 12 * 4
    assert plan(W.CONFIGS[1])["ctas"] == 32 * 8
    assert plan(W.CONFIGS[3])["ctas"] == SMS                  # one CTA per SM walks the 128 * 32 items
    assert plan(W.CONFIGS[3], flags=binding.FA_FLAG_NO_PERSISTENT)["ctas"] == 128 * 32


def test_table6_rows():
    got = {w.name: plan(w)["kernel"] for w, _ in W.TABLE6}
    assert got["gpt2_small_s2048"] == "fa_fwd_stream"          # 96 causal pairs: under a wave
    assert got["bert_base_s2048"] == "fa_fwd_pipelined"        # 192 equal tiles would make two waves
    assert got["llama3_8b_s2048"] == "fa_fwd_pair"
    assert got["qwen15_05b_s32768"] == "fa_fwd_stream"         # d = 64 with long items
    assert got["deepseek_67b_gqa_s4096"] == "fa_fwd_persistent"  # 1024 items of up to 32 K/V tiles, 7 per SM


def test_persistent_kernel_from_three_items_per_sm():
    kernel = lambda B, Hq, Hkv, S, causal: binding.fa_plan(SMS, B, Hq, Hkv, S, S, 128, 128, causal)["kernel"]
    # d = 128: the persistent kernel up to items of 128 K/V tiles (measured against the per-item kernel with the same
    # loop: 35 % ahead on 1-tile items, 9 % at 8, 3 % at 32, level at 128)
    assert kernel(4, 32, 8, 1024, True) == "fa_fwd_persistent"      # 512 items of up to 8 K/V tiles: 3.5 per SM
    assert kernel(4, 32, 32, 1024, True) == "fa_fwd_persistent"
    assert kernel(8, 32, 8, 512, True) == "fa_fwd_persistent"       # 512 items of up to 4 tiles
    assert kernel(4, 32, 8, 1024, False) == "fa_fwd_persistent"
    assert kernel(2, 32, 8, 1024, True) == "fa_fwd_pair"            # 256 items: under two per SM
    assert kernel(1, 32, 8, 2048, True) == "fa_fwd_pair"            # 256 items of up to 16 K/V tiles: under two per SM
    assert kernel(2, 32, 8, 2048, True) == "fa_fwd_persistent"      # 512 items of up to 16 K/V tiles
    assert kernel(4, 32, 32, 8192, True) == "fa_fwd_persistent"     # items of 64 K/V tiles
    assert kernel(1, 32, 8, 16384, True) == "fa_fwd_persistent"     # 2048 items of up to 128 K/V tiles
    assert kernel(1, 32, 8, 32768, True) == "fa_fwd_pair"           # items of 256 K/V tiles
    assert binding.fa_plan(SMS, 1, 32, 8, 32768, 32768, 128, 128, True, flags=binding.FA_FLAG_LEGACY_PAIR_KERNEL)["kernel"] == "fa_fwd_pipelined"
    assert binding.fa_plan(SMS, 8, 16, 16, 2048, 2048, 64, 64, True)["kernel"] == "fa_fwd_persistent"   # d = 64: up to 16 tiles
    assert binding.fa_plan(SMS, 4, 16, 16, 4096, 4096, 64, 64, True)["kernel"] == "fa_fwd_pipelined"


def test_decode_like_shapes_split_the_kv_range_on_the_stream_kernel():
    p = binding.fa_plan(SMS, 1, 32, 8, 128, 32768, 128, 128, False)
    assert p["kernel"] == "fa_fwd_stream" and p["kv_splits"] == 4 and p["ctas"] == 32 * 4
    p = binding.fa_plan(SMS, 8, 32, 32, 1, 8192, 128, 128, False)
    assert p["kernel"] == "fa_fwd_stream" and p["ctas"] == 256 * p["kv_splits"] and p["heads_per_tile"] == 1
    assert p["estimate_stream_us"] < p["estimate_pair_us"]


def test_few_queries_with_grouped_heads_share_a_query_tile():
    # 4 query heads per K/V head, one query each: all four in one tile, a quarter of the CTAs
    p = binding.fa_plan(SMS, 8, 32, 8, 1, 8192, 128, 128, False)
    assert p["kernel"] == "fa_fwd_stream" and p["heads_per_tile"] == 4 and p["ctas"] == 64 * p["kv_splits"]
    assert p["kv_splits"] == 2                                   # 64 items on 148 SMs
    # the largest divisor of the group size whose rows fit 128
    assert binding.fa_plan(SMS, 1, 16, 2, 16, 4096, 128, 128, True)["heads_per_tile"] == 8
    assert binding.fa_plan(SMS, 1, 16, 2, 20, 4096, 128, 128, True)["heads_per_tile"] == 4
    assert binding.fa_plan(SMS, 1, 12, 2, 33, 4096, 64, 64, True)["heads_per_tile"] == 3
    assert binding.fa_plan(SMS, 1, 12, 2, 64, 4096, 64, 64, True)["heads_per_tile"] == 2
    # not with more than 64 queries, one head per K/V head, or when switched off
    assert binding.fa_plan(SMS, 1, 12, 2, 65, 4096, 64, 64, True)["heads_per_tile"] == 1
    assert binding.fa_plan(SMS, 1, 12, 12, 16, 4096, 64, 64, True)["heads_per_tile"] == 1
    # packed batches of sequences (lengths on the device): packed heads; a small batch also splits the
    # K/V range (every CTA cuts its own sequence), a large one does not
    p = binding.fa_plan(SMS, 4, 16, 4, 16, 1024, 128, 128, True, varlen=True)
    assert p["kernel"] == "fa_fwd_stream" and p["heads_per_tile"] == 4 and p["kv_splits"] == 4 and p["ctas"] == 4 * 4 * 4
    p = binding.fa_plan(SMS, 64, 16, 4, 16, 1024, 128, 128, True, varlen=True)
    assert p["heads_per_tile"] == 4 and p["kv_splits"] == 1 and p["ctas"] == 64 * 4
    for flag in (binding.FA_FLAG_NO_HEAD_PACKING, binding.FA_FLAG_NO_STREAM_KERNEL, binding.FA_FLAG_SERIAL_KERNEL):
        assert binding.fa_plan(SMS, 8, 32, 8, 1, 8192, 128, 128, False, flags=flag)["heads_per_tile"] == 1


def test_flags_and_configuration_override_the_choice():
    w = W.CONFIGS[1]
    assert plan(w, flags=binding.FA_FLAG_STREAM_KERNEL)["kernel"] == "fa_fwd_stream_persistent"     # 512 one-tile items
    assert plan(w, flags=binding.FA_FLAG_STREAM_KERNEL | binding.FA_FLAG_NO_PERSISTENT)["kernel"] == "fa_fwd_stream"
    assert plan(w, flags=binding.FA_FLAG_FORCE_PERSISTENT | binding.FA_FLAG_NO_STREAM_KERNEL)["kernel"] == "fa_fwd_persistent"
    assert plan(w, flags=binding.FA_FLAG_SERIAL_KERNEL)["kernel"] == "fa_fwd_simple"
    assert plan(W.CONFIGS[0], flags=binding.FA_FLAG_NO_STREAM_KERNEL)["kernel"] == "fa_fwd_pipelined"
    # a forced split count is honoured as far as the scratch buffer holds the partials
    p = binding.fa_plan(SMS, 1, 32, 8, 128, 32768, 128, 128, False, kv_splits=7)
    assert p["kv_splits"] == 7
    p = binding.fa_plan(SMS, 1, 32, 8, 128, 32768, 128, 128, False, kv_splits=7, scratch_bytes=5 * 32 * 128 * 129 * 4)
    assert p["kv_splits"] == 5
    assert binding.fa_plan(SMS, 1, 32, 8, 128, 32768, 128, 128, False, kv_splits=1)["kv_splits"] == 1


def test_packed_batches_and_head_size_192():
    assert binding.fa_plan(SMS, 2, 16, 4, 1024, 1024, 128, 128, True, varlen=True)["kernel"] == "fa_fwd_pair"         # 128 items
    assert binding.fa_plan(SMS, 8, 16, 4, 1024, 1024, 128, 128, True, varlen=True)["kernel"] == "fa_fwd_persistent"   # 512 items of up to 8 K/V tiles
    assert binding.fa_plan(SMS, 4, 16, 4, 2048, 1024, 128, 128, True, varlen=True)["kernel"] == "fa_fwd_persistent"   # 512 items of up to 16
    assert binding.fa_plan(SMS, 4, 16, 4, 2048, 1024, 192, 128, True, varlen=True)["kernel"] == "fa_fwd_stream"
    assert binding.fa_plan(SMS, 1, 16, 16, 2048, 2048, 192, 128, True)["kernel"] == "fa_fwd_stream"


def test_argument_errors():
    with pytest.raises(binding.FaError):
        binding.fa_plan(SMS, 1, 3, 2, 128, 128, 128, 128, False)        # Hq not a multiple of Hkv
    with pytest.raises(binding.FaError):
        binding.fa_plan(SMS, 1, 2, 2, 128, 128, 96, 96, False)          # no kernel for this head size
    with pytest.raises(binding.FaError):
        binding.fa_plan(0, 1, 2, 2, 128, 128, 128, 128, False)


def test_packed_batches_of_many_short_sequences():
    plan = lambda B, Hq, Hkv, d, S=128, **kw: binding.fa_plan(SMS, B, Hq, Hkv, S, S, d, 128 if d == 192 else d, True, varlen=True, **kw)
    # many items per SM: the persistent kernel, heads of a group paired (one item per tile and pair of heads)
    p = plan(64, 32, 8, 128)
    assert p["kernel"] == "fa_fwd_persistent" and p["ctas"] == SMS and p["kv_splits"] == 1, p
    assert plan(8, 32, 8, 128, S=1024)["kernel"] == "fa_fwd_persistent"
    assert plan(8, 32, 8, 128, S=2048)["kernel"] == "fa_fwd_persistent"
    assert plan(1, 32, 8, 128, S=32768)["kernel"] == "fa_fwd_pair"      # items of 256 K/V tiles
    # without it: single tiles of two heads of a group share a CTA of the pair kernel
    p = plan(64, 32, 8, 128, flags=binding.FA_FLAG_NO_PERSISTENT)
    assert p["kernel"] == "fa_fwd_pair" and p["ctas"] == 64 * 16 and p["kv_splits"] == 1, p
    assert plan(4, 32, 8, 128)["kernel"] == "fa_fwd_stream"              # 128 items: under a wave of single tiles
    assert plan(64, 32, 32, 128, flags=binding.FA_FLAG_NO_PERSISTENT)["kernel"] == "fa_fwd_stream"   # nothing to pair
    assert plan(64, 32, 8, 192)["kernel"] == "fa_fwd_stream"             # 192/128 stays on the stream kernel
    assert plan(64, 32, 8, 128, flags=binding.FA_FLAG_NO_HEAD_PACKING | binding.FA_FLAG_NO_PERSISTENT)["kernel"] == "fa_fwd_stream"


def test_head_size_64_long_items():
    # The pair kernel at head size 64 keeps P in TMEM columns of its own and is ahead of the stream
    # kernel on causal items of up to 128 K/V tiles; without a mask, and on longer causal items, the
    # stream kernel stays ahead.
    kernel = lambda S, causal: binding.fa_plan(SMS, 1, 16, 16, S, S, 64, 64, causal)["kernel"]
    assert kernel(8192, True) == "fa_fwd_pipelined"
    assert kernel(16384, True) == "fa_fwd_pipelined"
    assert kernel(32768, True) == "fa_fwd_stream"
    assert kernel(8192, False) == "fa_fwd_stream"


def test_two_cta_kernel_is_used_only_where_it_applies():
    """Head size 64, packed batches and split-KV launches stay on the other kernels when the flag is set."""
    flags = binding.FA_FLAG_TWO_CTA_KERNEL
    assert binding.fa_plan(148, 1, 32, 8, 2048, 2048, 128, 128, True, flags=flags)["kernel"] == "fa_fwd_duo"
    assert binding.fa_plan(148, 1, 32, 8, 2048, 2048, 128, 128, True, flags=flags)["ctas"] == 2 * 16 * 16
    assert binding.fa_plan(148, 1, 128, 128, 4096, 4096, 192, 128, True, flags=flags)["kernel"] == "fa_fwd_duo"
    assert binding.fa_plan(148, 1, 16, 16, 2048, 2048, 64, 64, True, flags=flags)["kernel"] != "fa_fwd_duo"
    assert binding.fa_plan(148, 4, 16, 4, 1024, 1024, 128, 128, True, flags=flags, varlen=True)["kernel"] != "fa_fwd_duo"
    assert binding.fa_plan(148, 1, 32, 32, 128, 32768, 128, 128, False, flags=flags)["kernel"] != "fa_fwd_duo"   # split-KV


def test_quad_kernel_is_used_only_where_it_applies_and_picks_its_tiles_by_group_size():
    flags = binding.FA_FLAG_QUAD_KERNEL
    pl = binding.fa_plan(148, 1, 32, 8, 2048, 2048, 128, 128, True, flags=flags)
    assert pl["kernel"] == "fa_fwd_quad" and pl["ctas"] == 2 * 16 * 8            # four heads x one tile per cluster
    pl = binding.fa_plan(148, 1, 32, 16, 2048, 2048, 128, 128, True, flags=flags)
    assert pl["kernel"] == "fa_fwd_quad" and pl["ctas"] == 2 * 8 * 16            # two heads x two adjacent tiles
    pl = binding.fa_plan(148, 1, 128, 128, 4096 + 128, 4096 + 128, 192, 128, True, flags=flags)
    assert pl["kernel"] == "fa_fwd_quad" and pl["ctas"] == 2 * 9 * 128           # one head x four tiles, 33 tiles -> 9 clusters
    assert binding.fa_plan(148, 1, 16, 16, 2048, 2048, 64, 64, True, flags=flags)["kernel"] != "fa_fwd_quad"
    assert binding.fa_plan(148, 4, 16, 4, 1024, 1024, 128, 128, True, flags=flags, varlen=True)["kernel"] != "fa_fwd_quad"
    assert binding.fa_plan(148, 1, 32, 32, 128, 32768, 128, 128, False, flags=flags)["kernel"] != "fa_fwd_quad"   # split-KV


def test_persistent_stream_kernel_takes_short_one_tile_items_only():
    kernel = lambda B, H, S, causal, **kw: binding.fa_plan(SMS, B, H, H, S, S, 192, 128, causal, **kw)["kernel"]
    assert kernel(4, 128, 2048, True) == "fa_fwd_stream_persistent"       # 8192 items of up to 16 K/V tiles
    assert kernel(1, 128, 4096, True) == "fa_fwd_stream_persistent"       # up to 32
    assert kernel(1, 128, 8192, True) == "fa_fwd_stream"                  # longer items: no gain measured
    assert kernel(1, 8, 2048, True) == "fa_fwd_stream"                    # 128 items: under three per SM
    assert kernel(4, 128, 2048, True, flags=binding.FA_FLAG_NO_PERSISTENT) == "fa_fwd_stream"
    assert kernel(1, 128, 8192, True, flags=binding.FA_FLAG_FORCE_PERSISTENT | binding.FA_FLAG_STREAM_KERNEL) == "fa_fwd_stream_persistent"
    # packed batches and split-KV stay on the one-item kernel
    assert binding.fa_plan(SMS, 64, 128, 128, 512, 512, 192, 128, True, varlen=True)["kernel"] == "fa_fwd_stream"

