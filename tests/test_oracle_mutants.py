"""Do the pins bite?  Each case below plants one plausible mistake in a COPY of the oracle's C
source (a wrong rotation, a dropped term, a flipped comparison, a transposed layout ...),
builds it, and runs the matching pin file against it in a subprocess: the pins must fail.
Everything happens on the CPU; the real oracle is never modified."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "aibxo.c")
HDR = os.path.join(ROOT, "oracle", "aibxo.h")

# (name, pin file, text to find, replacement, which occurrence)
MUTANTS = [
    ("round_rotation", "test_oracle_hash.py", "acc = rotl64(acc, 31);", "acc = rotl64(acc, 30);", 0),
    ("prime2_digit", "test_oracle_hash.py", "0xC2B2AE3D27D4EB4FULL", "0xC2B2AE3D27D4EB4DULL", 0),
    ("merge_constant", "test_oracle_hash.py", "acc = acc * PRIME64_1 + PRIME64_4;\n  return acc;",
     "acc = acc * PRIME64_1 + PRIME64_3;\n  return acc;", 0),
    ("length_not_added", "test_oracle_hash.py", "acc += (uint64_t)len;", "", 0),
    ("avalanche_shift", "test_oracle_hash.py", "acc ^= acc >> 29;", "acc ^= acc >> 28;", 0),
    ("fourth_accumulator_sign", "test_oracle_hash.py", "uint64_t a4 = seed - PRIME64_1;",
     "uint64_t a4 = seed + PRIME64_1;", 0),
    ("chain_not_seeded_by_parent", "test_oracle_hash.py",
     "parent = aibxo_xxh64(msg, (size_t)block_tokens * 4, parent);",
     "parent = aibxo_xxh64(msg, (size_t)block_tokens * 4, root_seed);", 0),
    ("big_endian_tokens", "test_oracle_hash.py", "msg[4 * j + 0] = (uint8_t)(v);",
     "msg[4 * j + 0] = (uint8_t)(v >> 24);", 0),
    ("tail_word_rotation", "test_oracle_hash.py", "rotl64(acc, 23) * PRIME64_2 + PRIME64_3",
     "rotl64(acc, 22) * PRIME64_2 + PRIME64_3", 0),
    ("partial_block_hashed", "test_oracle_hash.py", "int64_t nblk = len / block_tokens;",
     "int64_t nblk = (len + block_tokens - 1) / block_tokens;", 0),
    ("insert_overwrites_mask", "test_oracle_index.py", "ix->e[w - 1].mask |= ix->e[i].mask;",
     "ix->e[w - 1].mask = ix->e[i].mask;", 0),
    ("insert_keeps_max_id", "test_oracle_index.py", "if (ix->e[i].id < ix->e[w - 1].id)",
     "if (ix->e[i].id > ix->e[w - 1].id)", 0),
    ("evict_keeps_named_bits", "test_oracle_index.py", "if (e) e->mask &= ~masks[i];",
     "if (e) e->mask &= masks[i];", 0),
    ("evict_reports_live_entries", "test_oracle_index.py",
     "freed[i] = (e && e->mask == 0) ? e->id : AIBXO_NO_BLOCK;",
     "freed[i] = (e && e->mask != 0) ? e->id : AIBXO_NO_BLOCK;", 0),
    ("all_ones_key_not_reserved", "test_oracle_index.py", "return k == 0ULL || k == ~0ULL;",
     "return k == 0ULL;", 0),
    ("touch_counts_twice_in_one_epoch", "test_oracle_index.py",
     "if (!e || e->epoch == epoch) continue;", "if (!e) continue;", 0),
    ("hot_after_one_touch", "test_oracle_index.py", "e->touches >= 2 ? (1u << 30)", "e->touches >= 1 ? (1u << 30)", 0),
    ("never_touched_looks_recent", "test_oracle_index.py",
     "ix->e[m].epoch = 0;", "ix->e[m].epoch = 5;", 0),
    ("export_drops_the_last_entry", "test_oracle_index.py",
     "for (uint64_t i = 0; i < ix->live && i < max_entries; ++i) {",
     "for (uint64_t i = 0; i + 1 < ix->live && i < max_entries; ++i) {", 0),
    ("rehash_accepts_too_small_a_table", "test_oracle_index.py",
     "if (ix->live > new_capacity) return AIBXO_ERR_FULL;", "", 0),
    ("pods_beyond_P_kept", "test_oracle_index.py", "ix->e[m].mask = masks[i] & all;",
     "ix->e[m].mask = masks[i];", 0),
    ("match_tests_wrong_pod", "test_oracle_match.py", "((e->mask >> p) & 1ULL) == 0) break;",
     "((e->mask >> (p + 1)) & 1ULL) == 0) break;", 0),
    ("match_ignores_pod_bit", "test_oracle_match.py",
     "if (!e || ((e->mask >> p) & 1ULL) == 0) break;", "if (!e) break;", 0),
    ("ids_after_a_hole", "test_oracle_match.py", "if (i < a) {\n          block_ids",
     "if (!key_reserved(h[i]) && find_entry(ix, h[i])) {\n          block_ids", 0),
    ("collect_keeps_duplicates", "test_oracle_match.py",
     "if (w == 0 || unique_ids[w - 1] != unique_ids[i])", "if (1)", 0),
    ("threshold_exclusive", "test_oracle_score.py", "100 * hit >= (int64_t)prm.threshold_pct * n_r",
     "100 * hit > (int64_t)prm.threshold_pct * n_r", 0),
    ("ties_to_highest_pod", "test_oracle_score.py", "arg == AIBXO_NO_POD || score > top",
     "arg == AIBXO_NO_POD || score >= top", 0),
    ("load_added", "test_oracle_score.py", "- (int64_t)prm.w_load * (int64_t)pod_load[p]",
     "+ (int64_t)prm.w_load * (int64_t)pod_load[p]", 0),
    ("ready_mask_ignored", "test_oracle_score.py", "if (((ready_mask >> p) & 1ULL) == 0) continue;",
     "", 0),
    ("threshold_on_tokens_not_blocks", "test_oracle_score.py",
     "100 * hit >= (int64_t)prm.threshold_pct * n_r", "100 * hit >= (int64_t)prm.threshold_pct * 16 * n_r", 0),
    ("assignment_forgets_the_increment", "test_oracle_score.py",
     "(uint32_t)pod_load[best_pod[r]] + (uint32_t)load_increment", "(uint32_t)pod_load[best_pod[r]]", 0),
    ("policy_picks_the_highest_figure", "test_oracle_policy.py",
     "if (arg == AIBXO_NO_POD || value[p] < value[arg]) arg = p;",
     "if (arg == AIBXO_NO_POD || value[p] > value[arg]) arg = p;", 0),
    ("policy_ties_to_the_last_pod", "test_oracle_policy.py",
     "if (arg == AIBXO_NO_POD || value[p] < value[arg]) arg = p;",
     "if (arg == AIBXO_NO_POD || value[p] <= value[arg]) arg = p;", 0),
    ("latency_ignores_the_queue", "test_oracle_policy.py",
     "const int32_t* b = policy == 4 ? metrics->serve_latency : NULL;",
     "const int32_t* b = NULL;", 0),
    ("latency_sum_wraps_in_32_bits", "test_oracle_policy.py",
     "value[p] = (int64_t)a[p] + (b ? (int64_t)b[p] : 0);",
     "value[p] = (int64_t)(int32_t)((uint32_t)a[p] + (b ? (uint32_t)b[p] : 0u));", 0),
    ("kv_policy_reads_requests", "test_oracle_policy.py",
     ": policy == 3 ? metrics->kv_usage", ": policy == 3 ? metrics->requests", 0),
    ("random_indexes_all_pods", "test_oracle_policy.py",
     "if ((ready_mask >> p) & 1ULL) ready[n++] = p;", "ready[n++] = p;", 0),
    ("prefix_policy_shortest_hit", "test_oracle_policy.py",
     "hit > arg_hit || (hit == arg_hit && value[p] < value[arg])",
     "hit < arg_hit || (hit == arg_hit && value[p] < value[arg])", 0),
    ("prefix_policy_ignores_requests_on_ties", "test_oracle_policy.py",
     "hit > arg_hit || (hit == arg_hit && value[p] < value[arg])", "hit > arg_hit", 0),
    ("prefix_policy_threshold_exclusive", "test_oracle_policy.py",
     "if (!(hit > 0 && 100 * hit >= (int64_t)threshold_pct * n_r)) continue;",
     "if (!(hit > 0 && 100 * hit > (int64_t)threshold_pct * n_r)) continue;", 0),
    ("prefix_policy_no_fallback", "test_oracle_policy.py",
     "if (arg == AIBXO_NO_POD) arg = lowest_ready(value, P, ready_mask);", "", 0),
    ("layer_major_as_block_major", "test_oracle_kv.py",
     "if (L->layout == 1) return (((int64_t)l * L->num_blocks + b) * 2 + kv) * half;",
     "if (L->layout == 1) return (((int64_t)b * L->num_layers + l) * 2 + kv) * half;", 0),
    ("split_kv_as_layer_major", "test_oracle_kv.py",
     "return (((int64_t)l * 2 + kv) * L->num_blocks + b) * half;",
     "return (((int64_t)l * L->num_blocks + b) * 2 + kv) * half;", 0),
    ("split_kv_planes_swapped", "test_oracle_kv.py",
     "return (((int64_t)l * 2 + kv) * L->num_blocks + b) * half;",
     "return (((int64_t)l * 2 + (1 - kv)) * L->num_blocks + b) * half;", 0),
    ("split_kv_layer_stride_of_one_plane", "test_oracle_kv.py",
     "return (((int64_t)l * 2 + kv) * L->num_blocks + b) * half;",
     "return (((int64_t)l + kv) * L->num_blocks + b) * half;", 0),
    ("buffer_layer_major", "test_oracle_kv.py",
     "return ((i * L->num_layers + l) * 2 + kv) * (tile_bytes(L) / 2);",
     "return ((l * L->num_blocks + i) * 2 + kv) * (tile_bytes(L) / 2);", 0),
    ("buffer_kv_outermost", "test_oracle_kv.py",
     "return ((i * L->num_layers + l) * 2 + kv) * (tile_bytes(L) / 2);",
     "return ((i * 2 + kv) * L->num_layers + l) * (tile_bytes(L) / 2);", 0),
    ("no_block_counts_as_error", "test_oracle_kv.py",
     "if (ids[i] == AIBXO_NO_BLOCK) continue;\n    if (ids[i] >= L->num_blocks) { ++nbad; continue; }\n    for (int32_t l = 0; l < L->num_layers; ++l)\n      for (int32_t kv = 0; kv < 2; ++kv)\n        memcpy((uint8_t*)buf",
     "if (ids[i] >= L->num_blocks) { ++nbad; continue; }\n    for (int32_t l = 0; l < L->num_layers; ++l)\n      for (int32_t kv = 0; kv < 2; ++kv)\n        memcpy((uint8_t*)buf", 0),
    ("scatter_copies_wrong_way", "test_oracle_kv.py",
     "memcpy((uint8_t*)pool + pool_offset(L, ids[i], l, kv),\n               (const uint8_t*)buf + buf_offset(L, i, l, kv), (size_t)half);",
     "memcpy((uint8_t*)buf + buf_offset(L, i, l, kv),\n               (const uint8_t*)pool + pool_offset(L, ids[i], l, kv), (size_t)half);", 0),
    ("inner_order_ignored_on_the_buffer_side", "test_oracle_kv.py",
     "uint8_t* brow = bhalf + row_offset(L, buf_inner, h, tok);",
     "uint8_t* brow = bhalf + row_offset(L, pool_inner, h, tok);", 0),
]


def _run_mutant(args):
    tmp, (name, pin_file, old, new, _) = args
    text = open(SRC).read()
    assert text.count(old) >= 1, "mutation site not found: " + name
    mutated = text.replace(old, new, 1)
    d = os.path.join(tmp, name)
    os.makedirs(d)
    with open(os.path.join(d, "aibxo.c"), "w") as f:
        f.write(mutated)
    with open(os.path.join(d, "aibxo.h"), "w") as f:
        f.write(open(HDR).read())
    lib = os.path.join(d, "libmutant.so")
    subprocess.check_call(["gcc", "-std=c99", "-O1", "-w", "-fPIC", "-shared",
                           os.path.join(d, "aibxo.c"), "-o", lib])
    env = dict(os.environ, AIBXO_LIB_OVERRIDE=lib, PYTHONDONTWRITEBYTECODE="1",
               OMP_NUM_THREADS="1", MKL_NUM_THREADS="1")
    try:
        r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                            os.path.join(ROOT, "tests", pin_file)],
                           cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT,
                           timeout=240)
    except subprocess.TimeoutExpired:
        return name, -9, "timed out (a broken copy that never returns is not a pass either)"
    return name, r.returncode, r.stdout.decode()[-400:]


def test_every_planted_mistake_is_caught(tmp_path):
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 2)) as pool:
        results = list(pool.map(_run_mutant, [(str(tmp_path), m) for m in MUTANTS]))
    survivors = [name for name, rc, _ in results if rc == 0]
    # exit 1 = a pin failed, a negative code = the broken copy crashed (also caught);
    # 2..5 are pytest's own errors and would mean the harness is not testing anything
    broken = [(name, rc, tail) for name, rc, tail in results if rc in (2, 3, 4, 5)]
    assert not broken, broken
    assert not survivors, "pins did not notice: %s" % survivors


def test_unmodified_copy_passes(tmp_path):
    """The harness itself: an untouched copy of the source passes a pin file."""
    name, rc, tail = _run_mutant((str(tmp_path), ("identity", "test_oracle_score.py",
                                                  "acc = rotl64(acc, 31);", "acc = rotl64(acc, 31);", 0)))
    assert rc == 0, tail


def test_pins_pass_on_a_sanitizer_build_of_the_oracle(tmp_path):
    """The unmodified oracle built with AddressSanitizer and UndefinedBehaviorSanitizer runs its
    pin files clean: no out-of-bounds access, no signed overflow, no misaligned load behind the
    results the GPU is compared with."""
    import shutil

    if shutil.which("gcc") is None:
        return
    lib = os.path.join(str(tmp_path), "libaibxo_san.so")
    try:
        subprocess.check_call(["gcc", "-std=c99", "-O1", "-g", "-fsanitize=address,undefined",
                               "-fno-sanitize-recover=undefined", "-fPIC", "-shared", SRC, "-o", lib],
                              stderr=subprocess.DEVNULL)
        asan = subprocess.check_output(["gcc", "-print-file-name=libasan.so"]).decode().strip()
    except (subprocess.CalledProcessError, OSError):
        return                                       # no sanitizer runtime on this machine
    if not os.path.isabs(asan) or not os.path.exists(asan):
        return
    env = dict(os.environ, AIBXO_LIB_OVERRIDE=lib, LD_PRELOAD=asan, PYTHONDONTWRITEBYTECODE="1",
               ASAN_OPTIONS="detect_leaks=0:abort_on_error=1", OMP_NUM_THREADS="1")
    files = ["test_oracle_hash.py", "test_oracle_index.py", "test_oracle_match.py",
             "test_oracle_score.py", "test_oracle_kv.py", "test_oracle_policy.py"]
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider"] +
                       [os.path.join(ROOT, "tests", f) for f in files],
                       cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, timeout=900)
    assert r.returncode == 0, r.stdout.decode()[-3000:]
