"""Seeded random argument sets for unpack + assemble (Section 4.3's consistency checks): a valid migration state
(prefix table, suffix blocks in arbitrary arrival order, fresh destination pages) and, for most cases, one or two
defects of the kinds the checks exist for.  Holds no expectation: the oracle says what each set deserves."""
import numpy as np

DEFECTS = ("none", "stale_epoch", "dst_out_of_range", "dst_negative", "dst_duplicate", "dst_in_prefix",
           "prefix_out_of_range", "prefix_duplicate", "logical_duplicate", "logical_below_prefix",
           "logical_beyond_end", "missing_block", "extra_block", "n_tokens_longer", "n_tokens_shorter")


def random_case(seed: int, num_blocks: int, block_size: int, max_blocks: int = 7):
    rng = np.random.default_rng(seed)
    n_prefix = int(rng.integers(0, max_blocks))
    n_suffix = int(rng.integers(0 if n_prefix else 1, max_blocks))
    phys = rng.permutation(num_blocks)[: n_prefix + n_suffix + 2]
    total = n_prefix + n_suffix
    # the last block may be partly filled; with no suffix the prefix ends on a block boundary
    n_tokens = total * block_size - (int(rng.integers(0, block_size)) if n_suffix else 0)
    order = rng.permutation(n_suffix)
    case = dict(prefix=[int(b) for b in phys[:n_prefix]],
                logical=[int(n_prefix + i) for i in order],
                dst=[int(phys[n_prefix + i]) for i in order],
                n=int(n_tokens), epoch=int(rng.integers(0, 5)))
    case["expected"] = case["epoch"]
    spare = [int(b) for b in phys[total:]]
    n_defects = int(rng.choice([0, 1, 1, 1, 2]))
    applied = []
    for _ in range(n_defects):
        kind = str(rng.choice(DEFECTS[1:]))
        applied.append(kind)
        dst, logical, prefix = case["dst"], case["logical"], case["prefix"]
        i = int(rng.integers(0, len(dst))) if dst else -1
        if kind == "stale_epoch":
            case["expected"] = case["epoch"] + 1
        elif kind == "dst_out_of_range" and dst:
            dst[i] = num_blocks + int(rng.integers(0, 3))
        elif kind == "dst_negative" and dst:
            dst[i] = -1 - int(rng.integers(0, 3))
        elif kind == "dst_duplicate" and len(dst) > 1:
            dst[i] = dst[(i + 1) % len(dst)]
        elif kind == "dst_in_prefix" and dst and prefix:
            dst[i] = prefix[int(rng.integers(0, len(prefix)))]
        elif kind == "prefix_out_of_range" and prefix:
            prefix[int(rng.integers(0, len(prefix)))] = num_blocks
        elif kind == "prefix_duplicate" and len(prefix) > 1:
            prefix[0] = prefix[1]
        elif kind == "logical_duplicate" and len(logical) > 1:
            logical[i] = logical[(i + 1) % len(logical)]
        elif kind == "logical_below_prefix" and logical and prefix:
            logical[i] = int(rng.integers(0, len(prefix)))
        elif kind == "logical_beyond_end" and logical:
            logical[i] = total + int(rng.integers(0, 3))
        elif kind == "missing_block" and dst:
            del dst[i], logical[i]
        elif kind == "extra_block":
            dst.append(spare[0])
            logical.append(total)
        elif kind == "n_tokens_longer":
            case["n"] = total * block_size + 1 + int(rng.integers(0, 2 * block_size))
        elif kind == "n_tokens_shorter" and total > 1:
            case["n"] = (total - 1) * block_size - int(rng.integers(0, block_size // 2))
        else:
            applied[-1] = "none"
    case["defects"] = applied
    return case
