"""B200-native AdLoCo hot path: norm test, switch-mode accumulation, outer step."""
