"""The pins must bite: plausible mistakes planted in a *copy* of the oracle's C source (on the CPU;
nothing here touches the GPU path) have to make at least one pin fail."""
import ctypes
import os
import subprocess

import pytest

import test_oracle_combine_pins as cpins
import test_oracle_order_pins as opins
import test_oracle_pair_pins as ppins
import test_oracle_pins as pins
import test_oracle_relay_pins as rpins
from oracle import mwo
from paper_2605_22428_b200 import workloads as wl

SRC = os.path.join(os.path.dirname(mwo.__file__), "mwo.c")

MUTATIONS = {
    "group-major blocks advance by one row": ("filled[r] += size;", "filled[r] += 1;"),
    "group-major ignores the position inside the group": ("group_dest_offset[(int64_t)g * Kd + i] + within;", "group_dest_offset[(int64_t)g * Kd + i];"),
    "group-major block copied from the start of the send buffer": ("const uint8_t *b_s = send_mw + (int64_t)group_offsets[g] * row_bytes;",
                                                                   "const uint8_t *b_s = send_mw;"),
    "expert index looks at the first slot only": ("for (int32_t k = 0; k < K; ++k) hit |= (topk_ids[(int64_t)t * K + k] == e);",
                                                  "hit = (topk_ids[(int64_t)t * K] == e);"),
    "expert index takes the slot of the first destination": ("if (dest_rank[(int64_t)t * Kd + i] == r) slot = dest_pos[(int64_t)t * Kd + i];",
                                                             "if (i == 0) slot = dest_pos[(int64_t)t * Kd + i];"),
    "expert index counts experts with a bad table entry": ("        if (r < 0 || r >= R) continue;\n        for (int32_t t = 0; t < T; ++t) {\n            int hit = 0;",
                                                           "        for (int32_t t = 0; t < T; ++t) {\n            int hit = 0;"),
    "binary32 combine rounds the product on its own": ("acc = fmaf(w, z, acc);", "{ volatile float prod = w * z; acc = prod + acc; }"),
    "binary32 combine walks the destinations downwards": (
        "float acc = 0.0f;\n            int any = 0;\n            for (int i = 0; i < Kd; ++i) {\n                const int32_t r = dest_rank[(int64_t)t * Kd + i];\n                if (r < 0) break;",
        "float acc = 0.0f;\n            int any = 0;\n            for (int i = Kd - 1; i >= 0; --i) {\n                const int32_t r = dest_rank[(int64_t)t * Kd + i];\n                if (r < 0) continue;"),
    "combine ignores the weights": ("acc += w * bf16_to_double(", "acc += bf16_to_double("),
    "combine truncates instead of rounding": ("double q = nearbyint(ldexp(a, 7 - ex));", "double q = floor(ldexp(a, 7 - ex));"),
    "combine reads the wrong slot": ("(int64_t)dest_pos[(int64_t)t * Kd + i] * row_bytes;\n                const double w",
                                     "(int64_t)(dest_pos[(int64_t)t * Kd + i] > 0 ? dest_pos[(int64_t)t * Kd + i] - 1 : 0) * row_bytes;\n                const double w"),
    "relay buffer in the receive buffer: the relay forwards a copy to itself again": (
        "if (r < 0 || r == h || mwo_next_hop(r, src_rank, ranks_per_server) != h) continue;\n                memcpy(region(recv_base, recv_stride_bytes, flat_rank_offsets, r, row_bytes) +\n                           (int64_t)flat_dest_pos[(int64_t)t * Kd + i] * row_bytes,\n                       held,",
        "if (r < 0 || mwo_next_hop(r, src_rank, ranks_per_server) != h) continue;\n                memcpy(region(recv_base, recv_stride_bytes, flat_rank_offsets, r, row_bytes) +\n                           (int64_t)(flat_dest_pos[(int64_t)t * Kd + i] + (r == h)) * row_bytes,\n                       held,"),
    "relay buffer in the receive buffer: forwarding always reads the hop area": (
        "const uint8_t *held = slot >= 0\n                ? region(recv_base, recv_stride_bytes, flat_rank_offsets, h, row_bytes) + (int64_t)slot * row_bytes\n                : hop_buf + (int64_t)q * row_bytes;",
        "const uint8_t *held = hop_buf + (int64_t)q * row_bytes;"),
    "relay buffer in the receive buffer: a pure relay's copy lands in the wrong hop row": (
        ": hop_buf + ((int64_t)hop_rank_offsets[h] + hop_dest_pos[(int64_t)t * Kd + i]) * row_bytes;",
        ": hop_buf + ((int64_t)hop_rank_offsets[h] + (hop_dest_pos[(int64_t)t * Kd + i] > 0 ? hop_dest_pos[(int64_t)t * Kd + i] - 1 : 0)) * row_bytes;"),
    "staged rows count every hop row": ("if (!is_dest) ++totals->staged_rows;", "++totals->staged_rows;"),
    "relay sends to rank 0 of the remote server": ("return (r / ranks_per_server) * ranks_per_server + src_rank % ranks_per_server;",
                                                   "return (r / ranks_per_server) * ranks_per_server;"),
    "paired allgather forwards the direct segment": ("relay_buf + ((int64_t)partner * copies + c) * relay_bytes, (size_t)relay_bytes);\n            ++k;",
                                                     "mine, (size_t)relay_bytes);\n            ++k;"),
    "split ignores the copies on the pair link": ("floor((double)shard_bytes * c * w_direct / (w_pair + c * w_direct));",
                                                  "floor((double)shard_bytes * w_direct / (w_pair + w_direct));"),
    "split with the two bandwidths exchanged": ("floor((double)shard_bytes * c * w_direct / (w_pair + c * w_direct));",
                                                "floor((double)shard_bytes * c * w_pair / (w_direct + c * w_pair));"),
    "bit index taken modulo 32": ("(uint64_t)1 << (r % 64)", "(uint64_t)1 << (r % 32)"),
    "always word 0": ("m[r / 64] |=", "m[0] |="),
    "padding treated as an error": ("if (id == -1) continue;                         /* padding slot            */", ""),
    "slot of the previous row": ("dest_pos[(int64_t)t * Kd + i] = rank_seen[r];",
                                 "dest_pos[(int64_t)t * Kd + i] = rank_seen[r] > 0 ? rank_seen[r] - 1 : 0;"),
    "rank offsets shifted": ("rank_offsets[r + 1] = rank_offsets[r] + rank_seen[r];",
                             "rank_offsets[r + 1] = rank_offsets[r] + rank_seen[r] - (r == 0 && rank_seen[r] > 0);"),
    "groups compared on the first word only": ("if (memcmp(group_mask + g * W, m, (size_t)W * sizeof(uint64_t)) == 0) break;",
                                               "if (memcmp(group_mask + g * W, m, sizeof(uint64_t)) == 0) break;"),
    "member order reversed in a group": ("int32_t row = group_offsets[g] + group_count[g]++;",
                                         "int32_t row = group_offsets[g + 1] - 1 - group_count[g]++;"),
    "deliver reads the wrong send row": ("send_mw + j * row_bytes, (size_t)row_bytes);\n        }\n    }\n}",
                                         "send_mw + (T_nonempty - 1 - j) * row_bytes, (size_t)row_bytes);\n        }\n    }\n}"),
    "unicast bytes count rows, not copies": ("totals->unicast_bytes = sent_copies * row_bytes;", "totals->unicast_bytes = sent_rows * row_bytes;"),
    "per-expert bytes deduplicated": ("++valid_slots;", "if (!(m[r / 64] >> (r % 64) & 1)) ++valid_slots;"),
    "metadata: one word instead of W": ("(int64_t)(8 * W);", "(int64_t)(8);"),
    "self copy counted as transmitted": ("if (src_rank >= 0 && (token_mask[(int64_t)t * W + src_rank / 64] >> (src_rank % 64) & 1)) --nd;", ""),
    "allgather metadata: one word instead of W": ("((shard_bytes + 4095) / 4096) * (8 * W);", "((shard_bytes + 4095) / 4096) * 8;"),
    "allgather metadata: per shard, not per packet": ("(int64_t)R * ((shard_bytes + 4095) / 4096) * (8 * W);", "(int64_t)R * (8 * W);"),
    "allgather metadata charged from the first rank on": ("totals->meta_bytes = (R <= 64 || R == 1) ? 0 :", "totals->meta_bytes = (R <= 1) ? 0 :"),
    "allgather transmits the self copy": ("if (dst_begin + d == i) continue;\n                memcpy(send_buf", "memcpy(send_buf"),
    "allgather unicast counts R copies": ("totals->unicast_bytes = (int64_t)R * (R - 1) * shard_bytes;", "totals->unicast_bytes = (int64_t)R * R * shard_bytes;"),
    "allgather shards concatenated in reverse": ("memcpy(recv_base + d * stride + (int64_t)i * shard_bytes,\n                       send_buf + (int64_t)i * shard_bytes",
                                                 "memcpy(recv_base + d * stride + (int64_t)(R - 1 - i) * shard_bytes,\n                       send_buf + (int64_t)i * shard_bytes"),
}


def run_pins():
    """A fast subset of the pins; raises AssertionError when the oracle is wrong."""
    for seed, (R, E, K) in enumerate([(3, 6, 2), (8, 32, 4), (9, 9, 3), (65, 130, 4), (2, 8, 5)]):
        inp = wl.make_random_dispatch(seed, T=29, K=K, E=E, R=R, H=8, pad_fraction=0.15 if seed % 2 else 0.0)
        pins.check_against_brute_force(inp, R)
    pins.test_brute_force_with_padding_duplicates_and_invalid_ids()
    pins.test_brute_force_source_inside_domain()
    pins.test_groups_differing_only_in_a_high_word()
    pins.test_paper_constants()
    pins.test_identical_and_all_distinct_tokens()
    for layout in (0, 1):
        pins.test_allgather_is_concatenate(layout, 5, 48, 1, 3)
        pins.test_allgather_is_concatenate(layout, 8, 64, 0, 8)
    pins.test_allgather_saved_closed_form_and_paper_example()
    pins.test_allgather_bitmap_overhead_beyond_64_ranks()
    cpins.test_one_hot_weights_select_one_destination(False)
    cpins.test_unit_weights_sum_small_integers_exactly()
    cpins.test_rounding_is_nearest_even_with_a_single_rounding()
    cpins.test_f32_mode_is_fused_multiply_add_in_rank_order_with_one_rounding(0, 8)
    cpins.test_f32_mode_does_not_round_the_product_before_the_addition()
    rpins.test_paper_example_four_local_four_remote()
    rpins.test_relay_brute_force(1, 12, 3, 7, 24, 4)
    ppins.test_every_rank_gets_its_domain_in_order(0, 8, 64, 32)
    ppins.test_split_by_bandwidth_ratio_lets_both_link_classes_finish_together(1, 4096 + 16, 8, 1.0, 7.0)
    opins.test_group_major_brute_force(1, 8, 32, 4, 0.2)
    opins.test_group_major_with_few_large_groups()
    opins.test_expert_index_brute_force(1, 8, 32, 4, 0.2, True)
    opins.test_expert_index_ignores_invalid_table_entries_and_ids()


def test_unmutated_oracle_passes_the_subset():
    run_pins()


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name, tmp_path, monkeypatch):
    old, new = MUTATIONS[name]
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutation anchor not found: {name}"
    mutated = tmp_path / "mwo_mut.c"
    mutated.write_text(text.replace(old, new, 1))
    lib_path = tmp_path / "libmwo_mut.so"
    subprocess.check_call(["gcc", "-O1", "-std=c11", "-shared", "-fPIC", "-w", "-o", str(lib_path), str(mutated), "-lm"])
    lib = ctypes.CDLL(str(lib_path))
    lib.mwo_plan.restype = ctypes.c_int
    lib.mwo_allgather.restype = ctypes.c_int
    lib.mwo_expert_index.restype = ctypes.c_int64
    for fn in ("mwo_pack_mw", "mwo_pack_uc", "mwo_deliver_mw", "mwo_deliver_uc", "mwo_deliver_definition"):
        getattr(lib, fn).restype = None
    monkeypatch.setattr(mwo, "_lib", lib)
    with pytest.raises(AssertionError):
        run_pins()
