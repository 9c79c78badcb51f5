"""Plain-Python oracle of the trie-based prefix index (Sec. 7.3 of the paper): insert, best-match
lookup, evict, pruning of nodes whose path probability is below epsilon.

TEST INFRASTRUCTURE ONLY.  It keeps the stored prefixes in a dictionary and answers every query by
brute force over all of them, so that it can be checked by eye against the definitions:
  * a stored prefix is kept up to the deepest node whose probability P(prefix) = prod_j P(x_j | x_<j)
    is at least epsilon (Def. 1 gives the edge weights; "pruned at nodes with probability below a
    threshold epsilon");
  * best match = the stored prefix with the longest common prefix with the query ("follow the path
    of the query until it diverges from all stored paths, and return the deepest stored ancestor");
    among several, the one whose stored token sequence is smallest in lexicographic order (a
    sequence that ends at the divergence node comes first), then the smallest id;
  * d_T of the match = -log2 P(common prefix) (Def. 2).
"""
import math


class TrieOracle:
    def __init__(self, epsilon=0.0):
        self.max_bits = math.inf if epsilon <= 0 else -math.log2(epsilon)
        self.stored = {}          # id -> (tuple of tokens kept, list of cumulative bits)

    def insert(self, ident, tokens, logp2):
        if ident in self.stored:
            raise KeyError(ident)
        kept, cum, bits = [], [0.0], 0.0
        for t, lp in zip(tokens, logp2):
            bits -= float(lp)
            if bits > self.max_bits:
                break
            kept.append(int(t)); cum.append(bits)
        self.stored[ident] = (tuple(kept), cum)
        return len(kept)

    def evict(self, ident):
        del self.stored[ident]

    def best_match(self, tokens):
        """Returns (id, lcp, d_T) or (-1, 0, 0.0) when nothing is stored."""
        best = None
        for ident, (seq, cum) in self.stored.items():
            m = 0
            while m < len(seq) and m < len(tokens) and seq[m] == int(tokens[m]):
                m += 1
            key = (-m, seq, ident)
            if best is None or key < best[0]:
                best = (key, ident, m, cum[m])
        if best is None:
            return -1, 0, 0.0
        return best[1], best[2], best[3]

    def n_nodes(self):
        """Distinct non-empty prefixes kept (= trie nodes without the root)."""
        nodes = set()
        for seq, _ in self.stored.values():
            for m in range(1, len(seq) + 1):
                nodes.add(seq[:m])
        return len(nodes)
